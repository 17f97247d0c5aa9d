"""GPU parity of the layer-wise regression step (Section 3.1, Eq. (w_b), Lemma 1) against the CPU checker:
the pre-activation gradient with loss and bias gradient, the tensor-core filter gradient, the SGD update, and
whole steps on a slim layer fitted to the feature map of conv -> BatchNorm -> Scale -> ReLU."""
import numpy as np
import pytest

import dr_synth as S
from util import LAYER_L2, LAYER_MAX, err_norms, to_dev_bf16, to_dev_f32, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dr():
    import paper_1708_04728_b200 as dr
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    return dr


@pytest.fixture(scope="module")
def F():
    import oracle.finetune as F
    return F


def workspace(nbytes, poison=True):
    import torch
    ws = torch.empty(max(nbytes, 4096) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    if poison:
        ws.fill_(0xFF)                       # NaN bit patterns: stale scratch must never reach a result
    return ws


def status_ok(dr):
    st, info = dr.dr_device_status()
    assert st == 0, f"device status {st} {info}"


def desc_of(dr, k, s, p, Cin, Cout, flags=0):
    return dr.dr_conv_desc(k=k, stride=s, pad=p, Cin=Cin, Cout=Cout, flags=flags, pool_k=3, pool_stride=2, pool_pad=1,
                           lrn_size=5, lrn_alpha=1e-4, lrn_beta=0.75, lrn_k=1.0, y_ldc=0, y_coff=0)


WGRAD_CASES = [
    # B, H, W, Cin, Cout, k, s, p
    (2, 14, 14, 64, 64, 3, 1, 1),       # 392 pixels: full pixel blocks (of 64 or 128) and a tail of 8
    (3, 17, 13, 96, 200, 3, 2, 1),      # channel tails on both sides (96 = 64 + 32, 200 = 128 + 72), stride 2
    (4, 8, 8, 128, 128, 1, 1, 0),       # 1x1: x read as a matrix
    (2, 9, 9, 64, 48, 5, 1, 2),         # 25 taps: seven column groups, the last with one unit; fewer than 64 filters
    (8, 28, 28, 64, 192, 3, 1, 1),      # 6272 pixels: several pixel ranges per output tile
    (1, 7, 7, 64, 8, 3, 1, 1),          # fewer pixels than one block
    (2, 14, 14, 528, 320, 3, 1, 1),     # 9 channel blocks per tap, the last of 16 channels; two column tiles (256 + 64)
    (2, 9, 9, 24, 20, 3, 1, 1),         # channel counts the tensor-core kernel does not take: the CUDA-core kernel
    (1, 16, 16, 3, 16, 7, 2, 3),        # three input channels, 7x7 / 2
]


@pytest.mark.parametrize("pair", [0, 1])
@pytest.mark.parametrize("B,H,W,Cin,Cout,k,s,p", WGRAD_CASES)
def test_wgrad_parity(dr, F, monkeypatch, B, H, W, Cin, Cout, k, s, p, pair):
    """Both tilings of the kernel on every case: one CTA per tile, and CTA pairs sharing a tile of twice the rows
    (forced here; the library picks by how much of the coarser tile a layer fills)."""
    import torch
    monkeypatch.setenv("DR_WGRAD_PAIR", str(pair))
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    x = S.round_bf16(S.normal(0, f"ft.x{B}.{H}.{Cin}", (B, H, W, Cin)))
    dz = S.round_bf16(S.normal(0, f"ft.dz{B}.{H}.{Cout}", (B, Ho, Wo, Cout)))
    d = desc_of(dr, k, s, p, Cin, Cout)
    need = dr.dr_conv_wgrad_workspace_bytes(d, B, H, W)
    ws = workspace(need)
    xd, dzd = to_dev_bf16(x), to_dev_bf16(dz)
    dw = torch.full((Cout, k, k, Cin), float("nan"), dtype=torch.float32, device="cuda")
    dr.dr_conv_wgrad(d, B, H, W, xd, dzd, dw, ws, ws.numel())
    status_ok(dr)
    ref = F.conv2d_wgrad(x, dz, k, s, p)
    got = to_host(dw)
    assert np.all(np.isfinite(got))
    mx, l2 = err_norms(got, ref)
    # exact products, float32 sums over at most a few thousand pixels
    assert mx <= 2e-5 and l2 <= 1e-5, f"max-rel {mx:.3e}, rel-L2 {l2:.3e}"
    dw2 = torch.zeros_like(dw)
    dr.dr_conv_wgrad(d, B, H, W, xd, dzd, dw2, ws, ws.numel())
    status_ok(dr)
    assert torch.equal(dw, dw2), "the filter gradient is not the same on a second run"


@pytest.mark.parametrize("H,Cin,Cout,k,s,p", [(14, 528, 512, 5, 1, 2),      # 4e merged 5x5: CTA pairs, 128-pixel stages
                                              (56, 64, 192, 3, 2, 1)])       # streamline conv2: single CTAs, 64-pixel stages
def test_wgrad_bench_size_sampled_filters(dr, F, H, Cin, Cout, k, s, p):
    """The layers and batch `bench.py --finetune` times, in the launch shape the library picks for them; the checker
    computes the gradient of a seeded sample of filters (its cost is proportional to the number of filters)."""
    import torch
    B = 256
    Ho = (H + 2 * p - k) // s + 1
    x = S.round_bf16(S.normal(0, f"ftb.x{H}", (B, H, H, Cin)).astype(np.float32))
    dz = S.round_bf16(S.normal(0, f"ftb.dz{H}", (B, Ho, Ho, Cout)).astype(np.float32))
    d = desc_of(dr, k, s, p, Cin, Cout)
    ws = workspace(dr.dr_conv_wgrad_workspace_bytes(d, B, H, H))
    dw = torch.full((Cout, k, k, Cin), float("nan"), dtype=torch.float32, device="cuda")
    dr.dr_conv_wgrad(d, B, H, H, to_dev_bf16(x), to_dev_bf16(dz), dw, ws, ws.numel())
    status_ok(dr)
    got = to_host(dw)
    assert np.all(np.isfinite(got))
    js = sorted(int(j) for j in S.stream(0, f"ftb.sample{H}").choice(Cout, size=4, replace=False)) + [0, Cout - 1]
    ref = F.conv2d_wgrad(x, dz[..., js], k, s, p)
    mx, l2 = err_norms(got[js], ref)
    assert mx <= 5e-5 and l2 <= 2e-5, f"max-rel {mx:.3e}, rel-L2 {l2:.3e}"      # float32 sums over 50 k - 200 k pixels
    # the rest: every filter's gradient has the size the sampled ones have (a dropped or doubled pixel range would not)
    norms = np.sqrt((got.reshape(Cout, -1) ** 2).sum(axis=1))
    assert norms.min() > 0.8 * np.median(norms) and norms.max() < 1.25 * np.median(norms)


@pytest.mark.parametrize("H,k,s,p", [(64, 7, 4, 3), (51, 11, 4, 0)])
def test_wgrad_of_a_strided_three_channel_stem(dr, F, H, k, s, p):
    """The stride-product stem of Section 3.1 (7x7/4 on RGB) and AlexNet's 11x11/4: the filter gradient is taken on the
    space-to-depth form (a stride-1 convolution over 64 channels) and gathered back to the original filter layout."""
    import torch
    B, C, Cout, Cp = 4, 3, 64, 64
    kp = (k + s - 1) // s
    Ho = (H + 2 * p - k) // s + 1
    x = S.round_bf16(S.normal(0, f"fts.x{k}", (B, H, H, C)))
    dz = S.round_bf16(S.normal(0, f"fts.dz{k}", (B, Ho, Ho, Cout)))
    xs = torch.zeros((B, Ho + kp - 1, Ho + kp - 1, Cp), dtype=torch.bfloat16, device="cuda")
    dr.dr_space_to_depth(B, H, H, C, k, s, p, Cp, to_dev_bf16(x), xs)
    d = desc_of(dr, kp, 1, 0, Cp, Cout)
    Hs = Ho + kp - 1
    ws = workspace(dr.dr_conv_wgrad_workspace_bytes(d, B, Hs, Hs))
    dws = torch.full((Cout, kp, kp, Cp), float("nan"), dtype=torch.float32, device="cuda")
    dr.dr_conv_wgrad(d, B, Hs, Hs, xs, to_dev_bf16(dz), dws, ws, ws.numel())
    dw = torch.full((Cout, k, k, C), float("nan"), dtype=torch.float32, device="cuda")
    dr.dr_s2d_filter_grad(Cout, k, C, s, Cp, dws, dw)
    status_ok(dr)
    mx, l2 = err_norms(to_host(dw), F.conv2d_wgrad(x, dz, k, s, p))
    assert mx <= 2e-5 and l2 <= 1e-5, f"max-rel {mx:.3e}, rel-L2 {l2:.3e}"


def test_wgrad_seeded_random_shapes(dr, F, monkeypatch):
    """Thirty seeded shapes around the tile edges: channel counts that are not multiples of 64, more than two column
    tiles, every kernel size and stride the networks use, pixel counts around the stage sizes; the tiling alternates
    between the library's choice, single CTAs and CTA pairs."""
    import torch
    r = S.stream(0, "ft.fuzz")
    for case in range(30):
        k = int(r.choice([1, 2, 3, 5, 7]))
        s_ = int(r.choice([1, 2]))
        p_ = int(r.integers(0, k // 2 + 1))
        Cin = int(r.choice([64, 72, 96, 128, 136, 200, 256]))
        Cout = int(r.choice([8, 40, 64, 120, 128, 136, 192, 256, 264, 320, 520, 600]))
        B = int(r.integers(1, 4))
        H = int(r.integers(max(k, 5), 19)); W = int(r.integers(max(k, 5), 19))
        Ho, Wo = (H + 2 * p_ - k) // s_ + 1, (W + 2 * p_ - k) // s_ + 1
        mode = ["", "0", "1"][case % 3]
        if mode:
            monkeypatch.setenv("DR_WGRAD_PAIR", mode)
        else:
            monkeypatch.delenv("DR_WGRAD_PAIR", raising=False)
        x = S.round_bf16(S.normal(0, f"fz.x{case}", (B, H, W, Cin)))
        dz = S.round_bf16(S.normal(0, f"fz.dz{case}", (B, Ho, Wo, Cout)))
        d = desc_of(dr, k, s_, p_, Cin, Cout)
        ws = workspace(dr.dr_conv_wgrad_workspace_bytes(d, B, H, W))
        dw = torch.full((Cout, k, k, Cin), float("nan"), dtype=torch.float32, device="cuda")
        dr.dr_conv_wgrad(d, B, H, W, to_dev_bf16(x), to_dev_bf16(dz), dw, ws, ws.numel())
        status_ok(dr)
        got = to_host(dw)
        what = f"case {case}: B{B} {H}x{W} Cin{Cin} Cout{Cout} k{k} s{s_} p{p_} pair='{mode}'"
        assert np.all(np.isfinite(got)), what
        mx, l2 = err_norms(got, F.conv2d_wgrad(x, dz, k, s_, p_))
        assert mx <= 2e-5 and l2 <= 1e-5, f"{what}: max-rel {mx:.3e}, rel-L2 {l2:.3e}"


def test_wgrad_degenerate(dr):
    import torch
    d = desc_of(dr, 3, 1, 1, 64, 64)
    dw = torch.full((64, 3, 3, 64), 5.0, dtype=torch.float32, device="cuda")
    ws = workspace(4096)
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    dr.dr_conv_wgrad(d, 0, 8, 8, x, x, dw, ws, ws.numel())           # empty batch: the gradient is zero
    assert float(dw.abs().sum()) == 0.0
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_wgrad(d, 4, 8, 8, x, x, dw, ws, 16)                # workspace too small
    assert e.value.status == dr.DR_ERR_WORKSPACE
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_wgrad(desc_of(dr, 3, 1, 1, 64, 64), 4, 8, 8, x, x, None, ws, ws.numel())
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    assert dr.dr_conv_wgrad_workspace_bytes(desc_of(dr, 3, 1, 1, 24, 64), 4, 8, 8) == 0     # CUDA-core kernel: no scratch


@pytest.mark.parametrize("B,H,W,C,relu", [(4, 9, 7, 64, 1), (4, 5, 5, 200, 0), (3, 14, 14, 192, 1), (2, 3, 3, 2048, 1), (1, 1, 1, 8, 1),
                                          (4, 6, 5, 20, 1), (2, 2, 2, 2056, 0)])       # the last two: the element-wise kernel
def test_regress_grad_parity(dr, F, B, H, W, C, relu):
    import torch
    y = S.round_bf16(np.maximum(S.normal(0, f"rg.y{B}.{C}", (B, H, W, C)), 0.0) if relu else S.normal(0, f"rg.y{B}.{C}", (B, H, W, C)))
    yt = S.round_bf16(np.abs(S.normal(0, f"rg.t{B}.{C}", (B, H, W, C))))
    ws = workspace(dr.dr_regress_workspace_bytes(C))
    dz = torch.full((B, H, W, C), float("nan"), dtype=torch.bfloat16, device="cuda")
    db = torch.full((C,), float("nan"), dtype=torch.float32, device="cuda")
    loss = torch.full((1,), float("nan"), dtype=torch.float32, device="cuda")
    dr.dr_regress_grad(B, H, W, C, to_dev_bf16(y), to_dev_bf16(yt), relu, dz, db, loss, ws, ws.numel())
    ref = F.grad_preactivation(y, yt, bool(relu))
    got = to_host(dz)
    if B & (B - 1) == 0:
        # 1/B is a power of two: the difference of two bf16 values and its scaling are exact in float32, so the
        # rounding to bf16 is the only rounding on both sides
        assert np.array_equal(got, S.round_bf16(ref))
    else:
        assert np.abs(got - ref).max() <= 2.0 ** -8 * np.abs(ref).max()
    assert np.array_equal(got == 0.0, ref == 0.0) or not relu
    assert abs(float(loss) - F.regression_loss(y, yt)) <= 1e-5 * F.regression_loss(y, yt)
    ref_db = F.bias_grad(got)                                            # the sums of the stored (rounded) dZ
    assert np.abs(to_host(db) - ref_db).max() <= 1e-5 * max(np.abs(ref_db).max(), 1e-30)


def test_sgd_update_parity(dr, F):
    import torch
    n = 100003
    w = S.normal(0, "sgd.w", (n,)).astype(np.float32)
    v = (0.1 * S.normal(0, "sgd.v", (n,))).astype(np.float32)
    g = S.normal(0, "sgd.g", (n,)).astype(np.float32)
    wd, vd, gd = to_dev_f32(w), to_dev_f32(v), to_dev_f32(g)
    shadow = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    dr.dr_sgd_update(n, wd, vd, gd, 0.01, 0.9, 5e-4, shadow)
    w_ref, v_ref = F.sgd_update(w, v, g, np.float32(0.01), np.float32(0.9), np.float32(5e-4))
    assert np.abs(to_host(vd) - v_ref).max() <= 1e-6 * np.abs(v_ref).max()
    assert np.abs(to_host(wd) - w_ref).max() <= 1e-6 * np.abs(w_ref).max()
    assert np.array_equal(to_host(shadow), S.round_bf16(to_host(wd)))   # the copy is the stored float32 value, rounded once


def test_regression_steps_on_a_folded_layer(dr, F):
    """A 3x3 slim layer is fitted to the output of conv -> BatchNorm -> Scale -> ReLU (Eq. (conv_bn_sl)): the
    gradients of one step against the checker fed the same stored forward output, then the loss trajectory of
    free-running steps on both sides."""
    import oracle as O
    import torch
    B, H, W, Cin, Cout, k, s, p = 4, 14, 14, 64, 96, 3, 1, 1
    x = S.round_bf16(S.normal(0, "ft.step.x", (B, H, W, Cin)))
    wt = S.he_normal(0, "ft.step.wt", Cout, k, Cin)
    mu, var = S.normal(0, "ft.mu", (Cout,), 0.1), S.uniform(0, "ft.var", (Cout,), 0.5, 1.5)
    gamma, beta = S.uniform(0, "ft.gamma", (Cout,), 0.5, 1.5), S.normal(0, "ft.beta", (Cout,), 0.1)
    yt = S.round_bf16(O.relu(O.scale(O.batchnorm(O.conv2d(x, wt, None, s, p), mu, var, 1.0, 1e-5), gamma, beta)))
    w0 = S.round_bf16(S.he_normal(0, "ft.step.w0", Cout, k, Cin))       # master and bf16 copy start equal
    b0 = np.zeros(Cout)
    lr, mom, decay = 0.001, 0.9, 1e-4
    d = desc_of(dr, k, s, p, Cin, Cout, dr.DR_BIAS | dr.DR_RELU)
    ws = workspace(dr.dr_regress_step_workspace_bytes(d, B, H, W), poison=False)
    ws.zero_()                                                           # the forward pass may keep tile counters there
    wd, bd = to_dev_f32(w0), to_dev_f32(b0)
    vw, vb = torch.zeros_like(wd), torch.zeros_like(bd)
    shadow = to_dev_bf16(w0)
    xd, ytd = to_dev_bf16(x), to_dev_bf16(yt)
    y = torch.zeros((B, H, W, Cout), dtype=torch.bfloat16, device="cuda")
    dz = torch.zeros_like(y)
    dw = torch.zeros((Cout, k, k, Cin), dtype=torch.float32, device="cuda")
    db = torch.zeros(Cout, dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    n0 = dr.dr_launch_count()

    def step():
        dr.dr_regress_step(d, B, H, W, xd, ytd, wd, bd, vw, vb, shadow, lr, mom, decay, y, dz, dw, db, loss, ws, ws.numel())
        return float(loss)

    l0 = step()
    status_ok(dr)
    assert dr.dr_launch_count() - n0 >= 7          # forward, gradient + its reduction, filter gradient + its reduction, two updates
    # one step, teacher-forced on the stored forward output
    y_gpu = to_host(y)
    y_ref = F.slim_forward(x, w0, b0, s, p)
    assert err_norms(y_gpu, y_ref)[1] <= LAYER_L2
    dz_ref = F.grad_preactivation(y_gpu, yt)
    mx, l2 = err_norms(to_host(dw), F.conv2d_wgrad(x, dz_ref, k, s, p))
    assert mx <= LAYER_MAX and l2 <= LAYER_L2, f"filter gradient: max-rel {mx:.3e}, rel-L2 {l2:.3e}"
    mx, l2 = err_norms(to_host(db), F.bias_grad(dz_ref))
    assert mx <= LAYER_MAX and l2 <= LAYER_L2, f"bias gradient: max-rel {mx:.3e}, rel-L2 {l2:.3e}"
    assert abs(l0 - F.regression_loss(y_gpu, yt)) <= 1e-4 * l0
    w1_ref, _ = F.sgd_update(w0, np.zeros_like(w0), to_host(dw), lr, mom, decay)
    assert err_norms(to_host(wd), w1_ref)[0] <= 1e-6
    assert np.array_equal(to_host(shadow), S.round_bf16(to_host(wd)))
    # free-running: the checker takes its own steps in float64 from the same start
    w, b, rvw, rvb = w0.copy(), b0.copy(), np.zeros_like(w0), np.zeros(Cout)
    ref_losses, gpu_losses = [], [l0]
    for i in range(12):
        w, b, rvw, rvb, l, _, _ = F.regression_step(x, yt, w, b, rvw, rvb, lr, mom, decay, s, p)
        ref_losses.append(l)
        if i < 11:
            gpu_losses.append(step())
    status_ok(dr)
    for i, (a, r) in enumerate(zip(gpu_losses, ref_losses)):
        assert abs(a - r) <= 2e-2 * r, f"step {i}: loss {a} vs {r}"
    assert gpu_losses[-1] < 0.7 * gpu_losses[0], gpu_losses


def _step_buffers(dr, B, Ho, Wo, Cin, Cout, k):
    import torch
    y = torch.zeros((B, Ho, Wo, Cout), dtype=torch.bfloat16, device="cuda")
    return (y, torch.zeros_like(y), torch.zeros((Cout, k, k, Cin), dtype=torch.float32, device="cuda"),
            torch.zeros(Cout, dtype=torch.float32, device="cuda"), torch.zeros(1, dtype=torch.float32, device="cuda"))


def test_shard_gradients_add_up_to_the_whole_step(dr, F):
    """A data-parallel step on one GPU: the mini-batch of 6 in uneven shards (4 + 2), each through dr_regress_shard_grads
    with the mini-batch's constant; the shards' dW, db and loss, added, are the checker's for the whole mini-batch."""
    B, H, W, Cin, Cout, k, s, p = 6, 14, 14, 64, 64, 3, 1, 1
    x = S.round_bf16(S.normal(5, "dp.x", (B, H, W, Cin)))
    yt = S.round_bf16(np.abs(S.normal(5, "dp.yt", (B, H, W, Cout))))
    w0 = S.round_bf16(S.he_normal(5, "dp.w", Cout, k, Cin)); b0 = S.normal(5, "dp.b", (Cout,), 0.05).astype(np.float32).astype(np.float64)
    d = desc_of(dr, k, s, p, Cin, Cout, dr.DR_BIAS | dr.DR_RELU)
    wbf, bd = to_dev_bf16(w0), to_dev_f32(b0)
    tot_dw, tot_db, tot_loss, ys = 0.0, 0.0, 0.0, []
    for a, e in ((0, 4), (4, 6)):
        n = e - a
        ws = workspace(dr.dr_regress_step_workspace_bytes(d, n, H, W), poison=False); ws.zero_()
        y, dz, dw, db, loss = _step_buffers(dr, n, H, W, Cin, Cout, k)
        dr.dr_regress_shard_grads(d, n, B, H, W, to_dev_bf16(x[a:e]), to_dev_bf16(yt[a:e]), wbf, bd, y, dz, dw, db, loss, ws, ws.numel())
        status_ok(dr)
        tot_dw = tot_dw + to_host(dw); tot_db = tot_db + to_host(db); tot_loss += float(loss)
        ys.append(to_host(y))
    y_gpu = np.concatenate(ys)
    dz_ref = F.grad_preactivation(y_gpu, yt)                      # teacher-forced on the stored forward output
    mx, l2 = err_norms(tot_dw, F.conv2d_wgrad(x, dz_ref, k, s, p))
    assert mx <= LAYER_MAX and l2 <= LAYER_L2, (mx, l2)
    mx, l2 = err_norms(tot_db, F.bias_grad(dz_ref))
    assert mx <= LAYER_MAX and l2 <= LAYER_L2, (mx, l2)
    assert abs(tot_loss - F.regression_loss(y_gpu, yt)) <= 1e-4 * tot_loss
    # free-running against the checker's own shard sums
    parts = [F.shard_gradients(x[a:e], yt[a:e], w0, b0, B, s, p) for a, e in ((0, 4), (4, 6))]
    assert err_norms(tot_dw, parts[0][0] + parts[1][0])[1] <= 2e-2
    with pytest.raises(dr.DrError) as e:                           # a shard cannot be larger than its mini-batch
        dr.dr_regress_shard_grads(d, 4, 2, H, W, wbf, wbf, wbf, bd, y, dz, dw, db, loss, ws, ws.numel())
    assert e.value.status == dr.DR_ERR_INVALID_ARG


def test_regression_step_on_channel_counts_the_tensor_kernels_do_not_take(dr, F):
    """A whole step on a layer with 24 input and 36 output channels (plain kernels throughout)."""
    import torch
    B, H, W, Cin, Cout, k, s, p = 3, 9, 11, 24, 36, 3, 1, 1
    x = S.round_bf16(S.normal(6, "odd.x", (B, H, W, Cin)))
    yt = S.round_bf16(np.abs(S.normal(6, "odd.yt", (B, H, W, Cout))))
    w0 = S.round_bf16(S.he_normal(6, "odd.w", Cout, k, Cin)); b0 = np.zeros(Cout)
    d = desc_of(dr, k, s, p, Cin, Cout, dr.DR_BIAS | dr.DR_RELU)
    ws = workspace(dr.dr_regress_step_workspace_bytes(d, B, H, W) + 256, poison=False); ws.zero_()
    wd, bd = to_dev_f32(w0), to_dev_f32(b0)
    vw, vb, shadow = torch.zeros_like(wd), torch.zeros_like(bd), to_dev_bf16(w0)
    y, dz, dw, db, loss = _step_buffers(dr, B, H, W, Cin, Cout, k)
    dr.dr_regress_step(d, B, H, W, to_dev_bf16(x), to_dev_bf16(yt), wd, bd, vw, vb, shadow, 1e-3, 0.9, 0.0, y, dz, dw, db, loss, ws, ws.numel())
    status_ok(dr)
    y_gpu = to_host(y)
    assert err_norms(y_gpu, F.slim_forward(x, w0, b0, s, p))[1] <= LAYER_L2
    dz_ref = F.grad_preactivation(y_gpu, yt)
    mx, l2 = err_norms(to_host(dw), F.conv2d_wgrad(x, dz_ref, k, s, p))
    assert mx <= LAYER_MAX and l2 <= LAYER_L2, (mx, l2)
    w1_ref, _ = F.sgd_update(w0, np.zeros_like(w0), to_host(dw), 1e-3, 0.9, 0.0)
    assert err_norms(to_host(wd), w1_ref)[0] <= 1e-6
