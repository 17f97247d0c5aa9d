"""GPU parity of dr_conv_slim / dr_inception_slim against the unfused CPU checker, per kernel path."""
import numpy as np
import pytest

import dr_synth as S
import dr_synth.params as P
from util import assert_layer_close, to_dev_bf16, to_dev_f32, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dr():
    import paper_1708_04728_b200 as dr
    yield dr
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)


@pytest.fixture(scope="module")
def O():
    import oracle
    return oracle


def oracle_slim_layer(O, x, w, b, k, s, p, flags, dr, residual=None, lrn=(5, 1e-4, 0.75, 1.0)):
    """The unfused layer sequence one slim layer stands for; returns (y, argmax or None)."""
    y = O.conv2d(x, w, b if flags & dr.DR_BIAS else None, s, p)
    arg = None
    if flags & dr.DR_RELU:
        y = O.relu(y)
    if flags & dr.DR_LRN and (flags & dr.DR_LRN_BEFORE_POOL or not flags & dr.DR_POOL):
        y = O.lrn(y, *lrn)
    if flags & dr.DR_POOL:
        y, arg = O.maxpool(y, 3, 2, 1)
        if flags & dr.DR_LRN and not flags & dr.DR_LRN_BEFORE_POOL:
            y = O.lrn(y, *lrn)
    if flags & dr.DR_RESIDUAL:
        y = O.add(y, residual)
        if flags & dr.DR_RELU_AFTER_RESIDUAL:
            y = O.relu(y)
    return y, arg


def run_conv(dr, x, w, b, k, s, p, flags, residual=None, ldc=0, coff=0, lrn=(5, 1e-4, 0.75, 1.0), want_argmax=False):
    import torch
    B, H, W, Cin = x.shape
    Cout = w.shape[0]
    d = dr.dr_conv_desc(k=k, stride=s, pad=p, Cin=Cin, Cout=Cout, flags=flags, pool_k=3, pool_stride=2, pool_pad=1,
                        lrn_size=lrn[0], lrn_alpha=lrn[1], lrn_beta=lrn[2], lrn_k=lrn[3], y_ldc=ldc, y_coff=coff)
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    if flags & dr.DR_POOL:
        Ho, Wo = (Ho - 1) // 2 + 1, (Wo - 1) // 2 + 1
    L = ldc or Cout
    dt = torch.float32 if flags & dr.DR_OUT_F32 else torch.bfloat16
    y = torch.full((B, Ho, Wo, L), 768.0, dtype=dt, device="cuda")      # canary outside the written slice
    arg = torch.full((B, Ho, Wo, Cout), -7, dtype=torch.int32, device="cuda") if want_argmax else None
    dr.dr_conv_slim(d, B, H, W, to_dev_bf16(x), to_dev_bf16(w), None if b is None else to_dev_f32(b),
                    None if residual is None else to_dev_bf16(residual), y, arg)
    st, info = dr.dr_device_status()
    assert st == 0, f"device status {st} {info}"
    yh = to_host(y)
    if L != Cout:
        mask = np.ones(L, bool); mask[coff:coff + Cout] = False
        assert np.all(yh[..., mask] == 768.0), "wrote outside its channel slice"
    return yh[..., coff:coff + Cout], (None if arg is None else arg.cpu().numpy())


def paths(dr):
    return [dr.DR_PATH_SIMT, dr.DR_PATH_UMMA_GATHER, dr.DR_PATH_UMMA_TMA]


def force(dr, path):
    dr.dr_set_conv_path(path)


# (B,H,W,Cin,Cout,k,s,p): several tiles, ragged tails in M, N and K
DIRECT_SHAPES = [
    (2, 9, 11, 64, 64, 3, 1, 1),      # M = 198: one full tile + tail
    (1, 28, 28, 192, 96, 1, 1, 0),    # 3a reducer
    (1, 14, 14, 96, 128, 3, 1, 1),
    (1, 12, 10, 48, 304, 5, 1, 2),    # two n-blocks of different width, K tail (48 of 64)
    (3, 7, 7, 160, 320, 3, 1, 1),     # 7x7 planes, tile spans images
    (2, 8, 8, 32, 40, 1, 2, 0),       # stride-2 1x1, Cout not a multiple of 16
    (1, 17, 13, 16, 16, 3, 2, 1),     # stride-2 3x3
    (2, 10, 10, 3, 64, 7, 2, 3),      # stem geometry, Cin = 3
    (5, 1, 1, 1024, 1000, 1, 1, 0),   # FC shape
    (2, 28, 28, 192, 128, 5, 1, 2),   # merged 5x5 of 3a
    (3, 14, 14, 480, 304, 5, 1, 2),   # merged 5x5 of 4a: n-blocks 160 + 144, 32-channel K tail
    (2, 7, 7, 832, 640, 5, 1, 2),     # merged 5x5 of 5b: three n-blocks, planes smaller than a tile
    (2, 16, 16, 256, 128, 1, 2, 0),   # ResNet stride-2 1x1 (first conv of a stage)
    (2, 15, 17, 64, 64, 3, 2, 1),     # stride-2 3x3, odd planes
    (1, 12, 12, 64, 32, 7, 1, 3),     # 7x7
    (2, 56, 56, 64, 256, 1, 1, 0),    # ResNet res2 expansion
]


@pytest.mark.parametrize("path", [1, 2, 3, 9])
@pytest.mark.parametrize("shape", DIRECT_SHAPES)
def test_conv_bias_relu(dr, O, path, shape):
    B, H, W, Cin, Cout, k, s, p = shape
    x = S.normal(10, "x", (B, H, W, Cin)); w = S.he_normal(10, "w", Cout, k, Cin); b = S.normal(10, "b", (Cout,), 0.1)
    force(dr, path)
    try:
        got, _ = run_conv(dr, x, w, b, k, s, p, dr.DR_BIAS | dr.DR_RELU)
    except dr.DrError as e:
        if e.status == dr.DR_ERR_UNSUPPORTED and path != dr.DR_PATH_SIMT:
            pytest.skip("path does not take this shape")
        raise
    assert dr.dr_last_conv_path() == path
    ref, _ = oracle_slim_layer(O, x, w, b, k, s, p, dr.DR_BIAS | dr.DR_RELU, dr)
    assert_layer_close(got, O.round_bf16(ref), f"path {path} {shape}")


# The patch-reuse kernel (path 9): tiles of whole padded image rows, every tap read out of one shared-memory patch.
# (B,H,W,Cin,Cout,k): planes of 28 / 14 / odd extents, image rows that do not fill the last tile of an image, an odd
# number of tiles (the second CTA of the last pair recomputes), channel tails in K (96, 480), one and two accumulator
# blocks (Cout <= 256 / > 256, equal and unequal halves), Cout not a multiple of 16.
QLIN_SHAPES = [
    (3, 28, 28, 192, 128, 5),     # merged 5x5 of 3a: 7 tiles per image, 21 tiles (odd)
    (2, 28, 28, 256, 288, 5),     # merged 5x5 of 3b: two blocks of 144
    (3, 14, 14, 480, 304, 5),     # merged 5x5 of 4a: blocks 160 + 144, 32-channel K tail, 2 tiles per image
    (2, 28, 28, 96, 128, 3),      # 3x3 of 3a: K tail (32 of 64)
    (5, 14, 14, 112, 224, 3),     # 3x3 of 4b
    (2, 13, 29, 64, 40, 5),       # odd plane, Cout not a multiple of 16
    (1, 30, 61, 64, 64, 3),       # wide rows: two image rows per tile
    (7, 9, 11, 128, 512, 5),      # two blocks of 256
    (2, 7, 7, 832, 384, 5),       # 7x7 planes: most of a tile is padding
]


@pytest.mark.parametrize("shape", QLIN_SHAPES)
@pytest.mark.parametrize("slice_", [False, True])
def test_conv_patch_reuse_kernel(dr, O, shape, slice_):
    B, H, W, Cin, Cout, k = shape
    x = S.normal(14, "x", (B, H, W, Cin)); w = S.he_normal(14, "w", Cout, k, Cin); b = S.normal(14, "b", (Cout,), 0.1)
    force(dr, dr.DR_PATH_UMMA_QLIN)
    ldc, coff = ((Cout + 72, 40) if slice_ else (0, 0))
    got, _ = run_conv(dr, x, w, b, k, 1, k // 2, dr.DR_BIAS | dr.DR_RELU, ldc=ldc, coff=coff)
    assert dr.dr_last_conv_path() == dr.DR_PATH_UMMA_QLIN
    ref, _ = oracle_slim_layer(O, x, w, b, k, 1, k // 2, dr.DR_BIAS | dr.DR_RELU, dr)
    assert_layer_close(got, O.round_bf16(ref), f"patch-reuse {shape}")
    again, _ = run_conv(dr, x, w, b, k, 1, k // 2, dr.DR_BIAS | dr.DR_RELU, ldc=ldc, coff=coff)
    assert np.array_equal(got, again)                                   # no atomics: bit-identical run to run


def test_conv_patch_reuse_kernel_residual_and_f32(dr, O):
    B, H, W, Cin, Cout, k = 2, 14, 14, 64, 96, 3
    x = S.normal(15, "x", (B, H, W, Cin)); w = S.he_normal(15, "w", Cout, k, Cin); b = S.normal(15, "b", (Cout,), 0.1)
    r = S.normal(15, "r", (B, H, W, Cout))
    force(dr, dr.DR_PATH_UMMA_QLIN)
    flags = dr.DR_BIAS | dr.DR_RESIDUAL | dr.DR_RELU_AFTER_RESIDUAL
    got, _ = run_conv(dr, x, w, b, k, 1, 1, flags, residual=r)
    ref, _ = oracle_slim_layer(O, x, w, b, k, 1, 1, flags, dr, residual=r)
    assert_layer_close(got, O.round_bf16(ref), "patch-reuse residual")
    got32, _ = run_conv(dr, x, w, b, k, 1, 1, dr.DR_BIAS | dr.DR_OUT_F32)
    ref32 = O.conv2d(x, w, b, 1, 1)
    assert np.abs(got32 - ref32).max() <= 2e-3 * np.abs(ref32).max()


@pytest.mark.parametrize("path", [1, 2, 3])
def test_conv_no_epilogue_f32_and_slice(dr, O, path):
    B, H, W, Cin, Cout, k, s, p = 2, 6, 7, 32, 48, 3, 1, 1
    x = S.normal(11, "x", (B, H, W, Cin)); w = S.he_normal(11, "w", Cout, k, Cin); b = S.normal(11, "b", (Cout,), 0.1)
    force(dr, path)
    try:
        got, _ = run_conv(dr, x, w, None, k, s, p, 0, ldc=96, coff=24)             # raw conv into a channel slice
        got32, _ = run_conv(dr, x, w, b, k, s, p, dr.DR_BIAS | dr.DR_OUT_F32)      # float32 store
    except dr.DrError as e:
        if e.status == dr.DR_ERR_UNSUPPORTED and path != dr.DR_PATH_SIMT:
            pytest.skip("path does not take this shape")
        raise
    ref = O.conv2d(x, w, None, s, p)
    assert_layer_close(got, O.round_bf16(ref), "slice")
    ref32 = O.conv2d(x, w, b, s, p)
    assert np.abs(got32 - ref32).max() <= 2e-3 * np.abs(ref32).max()   # bf16 products, fp32 accumulation, no output rounding


@pytest.mark.parametrize("path", [1, 2, 3])
def test_conv_residual_relu(dr, O, path):
    B, H, W, Cin, Cout = 2, 7, 7, 64, 256
    x = S.normal(12, "x", (B, H, W, Cin)); w = S.he_normal(12, "w", Cout, 1, Cin); b = S.normal(12, "b", (Cout,), 0.1)
    r = S.normal(12, "r", (B, H, W, Cout))
    flags = dr.DR_BIAS | dr.DR_RESIDUAL | dr.DR_RELU_AFTER_RESIDUAL
    force(dr, path)
    try:
        got, _ = run_conv(dr, x, w, b, 1, 1, 0, flags, residual=r)
    except dr.DrError as e:
        if e.status == dr.DR_ERR_UNSUPPORTED and path != dr.DR_PATH_SIMT:
            pytest.skip("path does not take this shape")
        raise
    ref, _ = oracle_slim_layer(O, x, w, b, 1, 1, 0, flags, dr, residual=r)
    assert_layer_close(got, O.round_bf16(ref), "residual")


def check_argmax(got_arg, ref_arg, pre_pool, ref_scale):
    """Integer parity where the decision is not a near-tie in the checker's own values."""
    B, Ho, Wo, Cc = pre_pool.shape
    flat = pre_pool.reshape(B, Ho * Wo, Cc)
    bad = got_arg != ref_arg
    n_bad = int(bad.sum())
    if n_bad == 0:
        return 0
    idx = np.argwhere(bad)
    excused = 0
    for n, ph, pw, c in idx:
        a, b_ = got_arg[n, ph, pw, c], ref_arg[n, ph, pw, c]
        assert 0 <= a < Ho * Wo, "argmax outside the plane"
        # the position chosen must lie inside the window and hold a value within tolerance of the maximum
        ah, aw = divmod(int(a), Wo)
        assert abs(ah - 2 * ph) <= 1 and abs(aw - 2 * pw) <= 1, "argmax outside its window"
        gap = flat[n, b_, c] - flat[n, a, c]
        assert 0 <= gap <= 1e-3 * ref_scale, f"argmax differs on a clear decision (gap {gap})"
        excused += 1
    return excused


# kernels that return the positions of the pooling maxima
ARGMAX_PATHS = (1, 2, 4, 5)

# fused pooling / LRN epilogues (Cout <= 256): (B,H,W,Cin,Cout,k,s,p, flags-name)
STAGED = [
    (1, 64, 64, 3, 64, 7, 2, 3, "pool_lrn"),        # the stem configuration: ReLU -> pool -> LRN
    (2, 20, 18, 64, 192, 3, 1, 1, "lrn_pool"),      # conv2 geometry: ReLU -> LRN -> pool
    (2, 13, 9, 32, 48, 3, 1, 1, "pool"),
    (1, 9, 12, 16, 32, 1, 1, 0, "lrn"),
    (2, 13, 11, 64, 96, 3, 1, 1, "lrn"),            # LRN without pooling on the TMA kernel: 3 chunks of 32 channels
    (1, 27, 27, 96, 256, 5, 1, 2, "lrn"),           # AlexNet conv2 as a dense layer: 256 channels, 32-channel K tail
    (3, 6, 5, 128, 48, 1, 1, 0, "lrn"),             # 16-channel tail chunk
    (1, 5, 5, 8, 16, 3, 1, 1, "pool"),              # plane smaller than one patch
    (3, 56, 56, 64, 192, 3, 1, 1, "lrn_pool"),      # GoogLeNet conv2 at its real plane size
    (2, 30, 26, 128, 64, 3, 1, 1, "pool"),          # two channel blocks per tap
    (2, 21, 19, 64, 96, 5, 1, 2, "pool_lrn"),       # 5x5, pool then LRN, float32 staging with 96 channels
    (2, 224, 224, 3, 64, 7, 2, 3, "pool_lrn"),      # GoogLeNet conv1 at full size
    (2, 70, 50, 3, 64, 7, 2, 3, "pool"),            # ResNet conv1 form (no LRN), ragged tiles
    (1, 38, 42, 3, 64, 7, 2, 3, "lrn_pool"),        # stem with LRN first
    (3, 100, 60, 3, 64, 7, 2, 3, "pool_lrn"),       # stem, ragged tiles in both directions, several images
    (120, 64, 64, 3, 64, 7, 2, 3, "pool_lrn"),      # stem, many images: long per-stream ranges that cross image boundaries
]


@pytest.mark.parametrize("path", [1, 2, 3, 4, 5, 7])
@pytest.mark.parametrize("case", STAGED)
def test_conv_fused_pool_lrn(dr, O, path, case):
    B, H, W, Cin, Cout, k, s, p, kind = case
    flags = dr.DR_BIAS | dr.DR_RELU | {"pool_lrn": dr.DR_POOL | dr.DR_LRN, "lrn_pool": dr.DR_POOL | dr.DR_LRN | dr.DR_LRN_BEFORE_POOL,
                                       "pool": dr.DR_POOL, "lrn": dr.DR_LRN}[kind]
    x = S.normal(0, "x", (B, H, W, Cin)); w = S.he_normal(0, "conv1.w", Cout, k, Cin); b = S.normal(0, "conv1.b", (Cout,), 0.01)
    lrn = (5, 1e-4, 0.75, 1.0) if kind == "pool_lrn" else (5, 0.05, 0.75, 1.0)      # second set makes LRN bite
    force(dr, path)
    try:
        got, arg = run_conv(dr, x, w, b, k, s, p, flags, lrn=lrn, want_argmax=bool(flags & dr.DR_POOL) and path in ARGMAX_PATHS)
    except dr.DrError as e:
        if e.status == dr.DR_ERR_UNSUPPORTED and path != dr.DR_PATH_SIMT:
            pytest.skip("path does not take this shape")
        raise
    ref, ref_arg = oracle_slim_layer(O, x, w, b, k, s, p, flags, dr, lrn=lrn)
    assert_layer_close(got, O.round_bf16(ref), f"{kind} path {path}")
    if arg is not None:
        pre = O.relu(O.conv2d(x, w, b, s, p))
        if flags & dr.DR_LRN_BEFORE_POOL:
            pre = O.lrn(pre, *lrn)
        excused = check_argmax(arg, ref_arg, pre, np.abs(pre).max())
        print(f"\n[argmax {kind} path {path} {case[:5]}] {excused} near-ties excused of {arg.size} positions ({100.0 * excused / arg.size:.3f} %)")
        assert excused <= 0.005 * arg.size + 8, f"{excused} near-ties of {arg.size}"


@pytest.mark.parametrize("path", [0, 1, 2, 4])
@pytest.mark.parametrize("kind", ["pool", "lrn_pool"])
def test_fused_pool_argmax_exact_ties_take_the_first_position(dr, O, path, kind):
    """Windows whose values are all exactly zero after ReLU (a large negative bias on some channels): the stored position
    must be the first of the window in row-major order, bit for bit, on every kernel that returns positions."""
    B, H, W, Cin, Cout, k, s, p = 2, 22, 18, 64, 64, 3, 1, 1
    flags = dr.DR_BIAS | dr.DR_RELU | dr.DR_POOL | (dr.DR_LRN | dr.DR_LRN_BEFORE_POOL if kind == "lrn_pool" else 0)
    x = S.normal(21, "x", (B, H, W, Cin)); w = S.he_normal(21, "w", Cout, k, Cin); b = S.normal(21, "b", (Cout,), 0.01).copy()
    dead = np.arange(0, Cout, 3)
    b[dead] = -64.0                                            # far below any pre-activation: ReLU gives exact zeros
    force(dr, path)
    try:
        got, arg = run_conv(dr, x, w, b, k, s, p, flags, want_argmax=True)
    except dr.DrError as e:
        if e.status == dr.DR_ERR_UNSUPPORTED and path != dr.DR_PATH_SIMT:
            pytest.skip("path does not take this shape")
        raise
    ref, ref_arg = oracle_slim_layer(O, x, w, b, k, s, p, flags, dr)
    assert np.all(ref[..., dead] == 0.0) and np.all(got[..., dead] == 0.0)
    assert np.array_equal(arg[..., dead], ref_arg[..., dead])
    # first position of a window: row max(2*ph - 1, 0), column max(2*pw - 1, 0)
    Hy, Wy = ref.shape[1], ref.shape[2]
    first = (np.maximum(2 * np.arange(Hy) - 1, 0)[:, None] * W + np.maximum(2 * np.arange(Wy) - 1, 0)[None, :]).astype(np.int32)
    assert np.array_equal(arg[0, :, :, dead[0]], first)


def test_inception_3a_config(dr, O):
    """Branch-slimmed inception module at the 3a shape: batch 8, 192x28x28."""
    import oracle.nets as N
    import torch
    params = P.inception_params(0, "3a")
    cin, c1, c3r, c3, _, c5, pp = S.INCEPTION_V1["3a"]
    cm = c1 + c5 + pp
    B = 8
    x = S.normal(0, "x", (B, 28, 28, cin))
    wm = torch.empty((cm, 5, 5, cin), dtype=torch.bfloat16, device="cuda")
    dr.dr_embed_filter(c1, cin, 1, 5, to_dev_bf16(params["3a.b1.w"]), 0, wm)
    dr.dr_embed_filter(c5, cin, 5, 5, to_dev_bf16(params["3a.b5.w"]), c1, wm)
    dr.dr_embed_filter(pp, cin, 3, 5, to_dev_bf16(params["3a.bp.w"]), c1 + c5, wm)
    bm = to_dev_f32(np.concatenate([params["3a.b1.b"], params["3a.b5.b"], params["3a.bp.b"]]))
    d = dr.dr_inception_desc(Cin=cin, c3r=c3r, c3=c3, cm=cm, pool_after=0)
    ws = torch.empty(dr.dr_inception_workspace_bytes(d, B, 28, 28), dtype=torch.uint8, device="cuda")
    y = torch.full((B, 28, 28, c3 + cm), 768.0, dtype=torch.bfloat16, device="cuda")
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    dr.dr_inception_slim(d, B, 28, 28, to_dev_bf16(x), [to_dev_bf16(params["3a.3x3r.w"]), to_dev_bf16(params["3a.3x3.w"]), wm],
                         [to_dev_f32(params["3a.3x3r.b"]), to_dev_f32(params["3a.3x3.b"]), bm], y, ws)
    assert dr.dr_device_status()[0] == 0
    got = to_host(y)
    out = N.run(N.inception_steps(params, "3a", "x"), x)
    assert_layer_close(got, out["3a"], "3a free-running")
    # teacher-forced 3x3: fed the reducer output the GPU stored
    red = to_host(ws[: B * 28 * 28 * c3r * 2].view(torch.bfloat16).reshape(B, 28, 28, c3r))
    assert_layer_close(red, out["3a.3x3r"], "3a.3x3r")
    forced = N.run(N.inception_steps(params, "3a", "x"), x, given={"3a.3x3r": red})
    assert_layer_close(got[..., :c3], forced["3a.3x3"], "3a.3x3 teacher-forced")
    assert_layer_close(got[..., c3:], forced["3a.m5"], "3a.m5")


def test_inception_with_pooling_after(dr, O):
    """pool_after: the module followed by the 3x3 / 2 max-pooling layer of inception 3b / 4e, odd plane (13 x 15)."""
    import oracle.nets as N
    import torch
    row = (64, 32, 64, 96, 16, 32, 32)                   # (Cin; c1, c3r, c3, c5r, c5, pp): a small module
    cin, c1, c3r, c3, _, c5, pp = row
    cm = c1 + c5 + pp
    params = P.inception_params(3, "m", {"m": row})
    B, H, W = 3, 13, 15
    x = S.normal(3, "x", (B, H, W, cin))
    wm = torch.empty((cm, 5, 5, cin), dtype=torch.bfloat16, device="cuda")
    dr.dr_embed_filter(c1, cin, 1, 5, to_dev_bf16(params["m.b1.w"]), 0, wm)
    dr.dr_embed_filter(c5, cin, 5, 5, to_dev_bf16(params["m.b5.w"]), c1, wm)
    dr.dr_embed_filter(pp, cin, 3, 5, to_dev_bf16(params["m.bp.w"]), c1 + c5, wm)
    bm = to_dev_f32(np.concatenate([params["m.b1.b"], params["m.b5.b"], params["m.bp.b"]]))
    d = dr.dr_inception_desc(Cin=cin, c3r=c3r, c3=c3, cm=cm, pool_after=1)
    d0 = dr.dr_inception_desc(Cin=cin, c3r=c3r, c3=c3, cm=cm, pool_after=0)
    need = dr.dr_inception_workspace_bytes(d, B, H, W)
    assert need >= dr.dr_inception_workspace_bytes(d0, B, H, W) + B * H * W * (c3 + cm) * 2
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    Hp, Wp = (H - 1) // 2 + 1, (W - 1) // 2 + 1
    y = torch.full((B, Hp, Wp, c3 + cm), 768.0, dtype=torch.bfloat16, device="cuda")
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    dr.dr_inception_slim(d, B, H, W, to_dev_bf16(x), [to_dev_bf16(params["m.3x3r.w"]), to_dev_bf16(params["m.3x3.w"]), wm],
                         [to_dev_f32(params["m.3x3r.b"]), to_dev_f32(params["m.3x3.b"]), bm], y, ws)
    assert dr.dr_device_status()[0] == 0
    full = N.run(N.inception_steps(params, "m", "x", table={"m": row}), x)["m"]
    want, _ = O.maxpool(O.round_bf16(full), 3, 2, 1)
    assert_layer_close(to_host(y), want, "module + pool")


def test_bounded_wait_reports_timeout_and_context_survives(dr, O):
    """A wait that can never be satisfied runs out after its limit, leaves DR_ERR_DEVICE_TIMEOUT in the status
    record, and the next layer on the same context still computes correctly."""
    assert dr.dr_device_status()[0] == 0
    dr.dr_selftest_wait_timeout(200000)                 # ~0.1 ms
    st, info = dr.dr_device_status()
    assert st == dr.DR_ERR_DEVICE_TIMEOUT and info[0] == dr.DR_ERR_DEVICE_TIMEOUT and info[1] == 99
    assert dr.dr_device_status()[0] == 0                # reading clears the record
    x = S.normal(20, "x", (1, 8, 8, 64)); w = S.he_normal(20, "w", 64, 3, 64); b = S.normal(20, "b", (64,), 0.1)
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    got, _ = run_conv(dr, x, w, b, 3, 1, 1, dr.DR_BIAS | dr.DR_RELU)
    ref, _ = oracle_slim_layer(O, x, w, b, 3, 1, 1, dr.DR_BIAS | dr.DR_RELU, dr)
    assert_layer_close(got, O.round_bf16(ref), "after timeout")
    with pytest.raises(dr.DrError):
        dr.dr_selftest_wait_timeout(0)


def test_conv_degenerate_shapes(dr, O):
    """Empty batch (nothing launched, canary untouched), a single output pixel, and a plane smaller than the filter's
    reach on every side (all taps but the centre ones fall on padding)."""
    import torch
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    d = dr.dr_conv_desc(k=3, stride=1, pad=1, Cin=64, Cout=64, flags=dr.DR_BIAS | dr.DR_RELU)
    y = torch.full((4, 4, 64), 768.0, dtype=torch.bfloat16, device="cuda")
    w = to_dev_bf16(S.he_normal(50, "w", 64, 3, 64)); b = to_dev_f32(S.normal(50, "b", (64,), 0.1))
    n0 = dr.dr_launch_count()
    dr.dr_conv_slim(d, 0, 4, 4, y, w, b, None, y)
    need = dr.dr_conv_workspace_bytes(d, 0, 4, 4)
    assert need == 0 and dr.dr_launch_count() == n0 and bool((y == 768.0).all())
    for shape in [(1, 1, 1, 64, 64, 3, 1, 1), (2, 2, 1, 128, 32, 5, 1, 2), (1, 1, 1, 64, 48, 7, 1, 3)]:
        B, H, W, Cin, Cout, k, s, p = shape
        x = S.normal(51, "x", (B, H, W, Cin)); wf = S.he_normal(51, "w", Cout, k, Cin); bf = S.normal(51, "b", (Cout,), 0.1)
        got, _ = run_conv(dr, x, wf, bf, k, s, p, dr.DR_BIAS | dr.DR_RELU)
        ref, _ = oracle_slim_layer(O, x, wf, bf, k, s, p, dr.DR_BIAS | dr.DR_RELU, dr)
        assert_layer_close(got, O.round_bf16(ref), f"degenerate {shape}")


@pytest.mark.parametrize("residual", [False, True])
def test_tma_epilogue_tail_rows_and_channel_slice(dr, O, residual, monkeypatch):
    """The shared-memory / TMA-store epilogue forced onto a small layer: a last tile with 41 of 128 rows (the tensor map
    clips the rest), a 64 + 32 column split (the 32 go out through the direct stores), a channel slice of a wider
    tensor (nothing outside it may be written), and the residual variant (boxes loaded by TMA, added in place)."""
    monkeypatch.setenv("DR_TMA_STORE_EP", "2")
    dr.dr_set_conv_path(dr.DR_PATH_UMMA_TMA)
    B, H, W, Cin = 3, 9, 11, 64
    Cout = 128 if residual else 96
    x = S.normal(60, "x", (B, H, W, Cin)); w = S.he_normal(60, "w", Cout, 1, Cin); b = S.normal(60, "b", (Cout,), 0.1)
    if residual:
        r = S.normal(60, "r", (B, H, W, Cout))
        flags = dr.DR_BIAS | dr.DR_RESIDUAL | dr.DR_RELU_AFTER_RESIDUAL
        got, _ = run_conv(dr, x, w, b, 1, 1, 0, flags, residual=r, ldc=256, coff=64)
        ref = O.relu(O.add(O.conv2d(x, w, b, 1, 0), r))
    else:
        got, _ = run_conv(dr, x, w, b, 1, 1, 0, dr.DR_BIAS | dr.DR_RELU, ldc=256, coff=64)
        ref = O.relu(O.conv2d(x, w, b, 1, 0))
    assert_layer_close(got, O.round_bf16(ref), "TMA epilogue")
    monkeypatch.setenv("DR_TMA_STORE_EP", "0")
    if residual:
        got0, _ = run_conv(dr, x, w, b, 1, 1, 0, flags, residual=r, ldc=256, coff=64)
    else:
        got0, _ = run_conv(dr, x, w, b, 1, 1, 0, dr.DR_BIAS | dr.DR_RELU, ldc=256, coff=64)
    assert np.array_equal(got, got0)                 # same arithmetic, one rounding: bit-identical to the direct stores
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
