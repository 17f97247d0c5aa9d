"""Host-side checks of the C-ABI library: it loads, exports every declared symbol, validates
arguments before touching the device, and builds the two networks' layer lists (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def dr():
    import __graft_entry__
    __graft_entry__.build_cuda()
    import paper_1708_04728_b200 as dr
    return dr


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dr_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(dr):
    lib = C.CDLL(dr.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 30
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/dr.h but not exported"
    assert set(dr.EXPORTS) == set(names), set(dr.EXPORTS) ^ set(names)


def test_strerror(dr):
    assert dr.dr_strerror(0) == "ok"
    for code in range(-6, 0):
        assert dr.dr_strerror(code) not in ("ok", "unknown status")
    assert dr.dr_strerror(-99) == "unknown status"


def test_conv_validation_rejects_before_launch(dr):
    d = dr.dr_conv_desc(k=3, stride=1, pad=1, Cin=16, Cout=16, flags=dr.DR_BIAS)
    n0 = dr.dr_launch_count()
    with pytest.raises(dr.DrError) as e:       # null pointers
        dr.dr_conv_slim(d, 1, 8, 8, None, None, None, None, None, None, 0)
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    with pytest.raises(dr.DrError) as e:       # bias flag without bias
        dr.dr_conv_slim(d, 1, 8, 8, 256, 256, None, None, 256, None, 0)
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    with pytest.raises(dr.DrError) as e:       # misaligned pointer
        dr.dr_conv_slim(d, 1, 8, 8, 260, 256, 256, None, 256, None, 0)
    assert e.value.status == dr.DR_ERR_ALIGNMENT
    d.flags = dr.DR_POOL | dr.DR_RESIDUAL
    d.pool_k, d.pool_stride, d.pool_pad = 3, 2, 1
    with pytest.raises(dr.DrError) as e:       # pooling together with a residual is not built
        dr.dr_conv_slim(d, 1, 8, 8, 256, 256, None, 256, 256, None, 0)
    assert e.value.status == dr.DR_ERR_UNSUPPORTED
    d.flags = dr.DR_POOL
    d.pool_k = 2
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_slim(d, 1, 8, 8, 256, 256, None, None, 256, None, 0)
    assert e.value.status == dr.DR_ERR_UNSUPPORTED
    d = dr.dr_conv_desc(k=3, stride=1, pad=1, Cin=16, Cout=16, flags=0, y_ldc=20, y_coff=0)
    with pytest.raises(dr.DrError) as e:       # channel stride not a multiple of 8
        dr.dr_conv_slim(d, 1, 8, 8, 256, 256, None, None, 256, None, 0)
    assert e.value.status == dr.DR_ERR_ALIGNMENT
    d = dr.dr_conv_desc(k=9, stride=1, pad=0, Cin=16, Cout=16, flags=0)
    with pytest.raises(dr.DrError) as e:       # kernel larger than the padded plane
        dr.dr_conv_slim(d, 1, 8, 8, 256, 256, None, None, 256, None, 0)
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    assert dr.dr_launch_count() == n0


def test_conv_workspace_query_and_validation(dr):
    """Host-only: which layers want split-K scratch, and argument checks of dr_conv_slim_ws."""
    d = dr.dr_conv_desc(k=5, stride=1, pad=2, Cin=832, Cout=640, flags=dr.DR_BIAS | dr.DR_RELU)
    small, large = dr.dr_conv_workspace_bytes(d, 1, 7, 7), dr.dr_conv_workspace_bytes(d, 256, 7, 7)
    assert small > dr.DR_CONV_WS_COUNTER_BYTES and large == 0
    assert small < 64 << 20
    d3 = dr.dr_conv_desc(k=7, stride=2, pad=3, Cin=3, Cout=64, flags=dr.DR_BIAS)      # stem: never split
    assert dr.dr_conv_workspace_bytes(d3, 1, 224, 224) == 0
    n0 = dr.dr_launch_count()
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_slim_ws(d, 1, 7, 7, 256, 256, 256, None, 256, None, 260, 1 << 20, 0)   # workspace not 256-byte aligned
    assert e.value.status == dr.DR_ERR_ALIGNMENT
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_slim_ws(d, 1, 7, 7, None, 256, 256, None, 256, None, 256, 1 << 20, 0)
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    assert dr.dr_launch_count() == n0


def test_regression_entry_points_validate_before_launch(dr):
    """Host-only: workspace queries and argument checks of the layer-wise regression calls (Eq. (w_b))."""
    d = dr.dr_conv_desc(k=3, stride=1, pad=1, Cin=64, Cout=192, flags=dr.DR_BIAS | dr.DR_RELU)
    wg = dr.dr_conv_wgrad_workspace_bytes(d, 256, 28, 28)
    assert wg % 256 == 0 and wg >= 192 * 576 * 4 and wg % (192 * 576 * 4) == 0      # whole partial copies of the gradient
    assert dr.dr_conv_wgrad_workspace_bytes(d, 0, 28, 28) == 0
    assert dr.dr_regress_workspace_bytes(192) >= 193 * 4
    assert dr.dr_regress_step_workspace_bytes(d, 256, 28, 28) >= wg + dr.dr_regress_workspace_bytes(192)
    n0 = dr.dr_launch_count()
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_wgrad(d, 4, 8, 8, 256, 256, 256, 260, 1 << 30, 0)                  # workspace not 256-byte aligned
    assert e.value.status == dr.DR_ERR_ALIGNMENT
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_wgrad(d, 4, 8, 8, None, 256, 256, 256, 1 << 30, 0)
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    with pytest.raises(dr.DrError) as e:
        dr.dr_regress_grad(4, 8, 8, 20, 256, 256, 1, 256, 256, None, 260, 1 << 20, 0)   # workspace not 256-byte aligned
    assert e.value.status == dr.DR_ERR_ALIGNMENT
    with pytest.raises(dr.DrError) as e:
        dr.dr_regress_grad(4, 8, 8, 64, 256, 256, 1, 256, 256, None, 256, 16, 0)
    assert e.value.status == dr.DR_ERR_WORKSPACE
    with pytest.raises(dr.DrError) as e:
        dr.dr_sgd_update(16, None, 256, 256, 0.1, 0.9, 0.0, None, 0)
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    dp = dr.dr_conv_desc(k=3, stride=1, pad=1, Cin=64, Cout=192, flags=dr.DR_BIAS | dr.DR_RELU | dr.DR_POOL, pool_k=3, pool_stride=2, pool_pad=1)
    with pytest.raises(dr.DrError) as e:                                               # only bias / ReLU layers are re-learned
        dr.dr_regress_step(dp, 4, 8, 8, 256, 256, 256, 256, 256, 256, 256, 0.1, 0.9, 0.0, 256, 256, 256, 256, None, 256, 1 << 30, 0)
    assert e.value.status == dr.DR_ERR_UNSUPPORTED
    assert dr.dr_launch_count() == n0


def test_non_tensor_validation(dr):
    n0 = dr.dr_launch_count()
    for call in (lambda: dr.dr_relu(16, None, 256, 0),
                 lambda: dr.dr_maxpool(1, 8, 8, 8, 3, 2, 1, None, 256, None, 0),
                 lambda: dr.dr_lrn(1, 8, 8, 8, 4, 1e-4, 0.75, 1.0, 256, 256, 0),      # even window
                 lambda: dr.dr_bn(1, 8, 8, 8, 256, 256, 256, 0.0, 0.0, None, None, 256, 0),  # m = 0
                 lambda: dr.dr_concat(4, 8, 256, 8, 8, 256, 0),                        # slice outside ldc
                 lambda: dr.dr_fold_bn(0, 9, 256, None, 256, 256, 1.0, 0.0, 256, 256, 256, 256, 0)):
        with pytest.raises(dr.DrError) as e:
            call()
        assert e.value.status == dr.DR_ERR_INVALID_ARG
    with pytest.raises(dr.DrError) as e:
        dr.dr_relu(16, 257, 256, 0)
    assert e.value.status == dr.DR_ERR_ALIGNMENT
    assert dr.dr_launch_count() == n0


def test_googlenet_layer_lists(dr):
    slim = dr.Net(dr.DR_ARCH_GOOGLENET, dr.DR_MODE_SLIM, 2)
    uns = dr.Net(dr.DR_ARCH_GOOGLENET, dr.DR_MODE_UNSLIMMED, 2)
    names = [slim.dr_net_layer_info(i)["name"] for i in range(slim.dr_net_num_layers())]
    # 3 stem convs + 9 modules x 3 convs + 2 pools + avg-pool + fc
    assert len(names) == 3 + 27 + 2 + 1 + 1
    assert names[:3] == ["conv1", "conv2r", "conv2"] and names[-2:] == ["avgpool", "fc"]
    assert sum(slim.dr_net_layer_info(i)["kind"] == 0 for i in range(len(names))) == 31
    li = {slim.dr_net_layer_info(i)["name"]: slim.dr_net_layer_info(i) for i in range(len(names))}
    assert li["conv1"]["dims"] == (2, 56, 56, 64) and li["conv2"]["dims"] == (2, 28, 28, 192)
    assert li["3a.3x3"]["dims"] == (2, 28, 28, 128) and (li["3a.3x3"]["ldc"], li["3a.3x3"]["coff"]) == (256, 0)
    assert li["3a.m5"]["dims"] == (2, 28, 28, 128) and (li["3a.m5"]["ldc"], li["3a.m5"]["coff"]) == (256, 128)
    assert li["5b.m5"]["dims"] == (2, 7, 7, 640) and li["5b.m5"]["ldc"] == 1024
    assert li["fc"]["dims"] == (2, 1, 1, 1000) and li["fc"]["is_f32"]
    # dense merged 5x5 FLOPs: 2*M*N*K
    assert li["3a.m5"]["flops"] == 2.0 * (2 * 28 * 28) * 128 * (25 * 192)
    total = sum(v["flops"] for v in li.values()) / 2
    assert abs(total / 1e9 - 16.64) < 0.02          # GFLOP per image of the branch-slimmed form
    # both modes take the same parameter list
    ps = [slim.dr_net_param_spec(i) for i in range(slim.dr_net_num_params())]
    pu = [uns.dr_net_param_spec(i) for i in range(uns.dr_net_num_params())]
    assert ps == pu and len(ps) == 2 * (3 + 9 * 5 + 1)
    n_uns = uns.dr_net_num_layers()
    kinds = [uns.dr_net_layer_info(i)["kind"] for i in range(n_uns)]
    assert kinds.count(0) == 3 + 9 * 5 + 1 and n_uns > 2 * len(names)
    assert slim.dr_net_workspace_bytes() > 0 and uns.dr_net_activation_bytes() > slim.dr_net_activation_bytes()
    with pytest.raises(dr.DrError) as e:      # forward before prepare
        slim.dr_net_forward(256, 256, 256, 0)
    assert e.value.status == dr.DR_ERR_WORKSPACE


def test_googlenet_paper_form_layer_list(dr):
    net = dr.Net(dr.DR_ARCH_GOOGLENET_PAPER, dr.DR_MODE_SLIM, 1)
    infos = {net.dr_net_layer_info(i)["name"]: net.dr_net_layer_info(i) for i in range(net.dr_net_num_layers())}
    assert net.dr_net_num_layers() == 3 + 9 * 4 + 2 + 1 + 1
    # the numbers Section 3.2 gives for inception_3a: reducer 96 -> 48, 3x3 128 -> 192, 5x5 32 -> 64
    # the 48-channel reducer is stored in a 64-channel tensor (the rest zeros: the 3x3 kernel reads channels in 64s);
    # its work is counted for 48 channels, and so is the 3x3's
    assert infos["3a.p3r"]["dims"] == (1, 28, 28, 64)
    assert infos["3a.p3r"]["flops"] == 2.0 * 784 * 48 * 192 and infos["3a.p3"]["flops"] == 2.0 * 784 * 192 * 9 * 48
    assert infos["3a.p5r"]["dims"] == (1, 28, 28, 64) and infos["3a.p5"]["flops"] == 2.0 * 784 * 64 * 25 * 16
    assert infos["3a.p3"]["dims"] == (1, 28, 28, 192) and (infos["3a.p3"]["ldc"], infos["3a.p3"]["coff"]) == (256, 0)
    assert infos["3a.p5"]["dims"] == (1, 28, 28, 64) and (infos["3a.p5"]["ldc"], infos["3a.p5"]["coff"]) == (256, 192)
    assert infos["5b.p5"]["ldc"] == 1024
    gflop = sum(v["flops"] for v in infos.values()) / 1e9
    assert 1.5 < gflop < 3.5          # far fewer FLOPs than the merged-5x5 form (16.6)


def test_googlenet_streamline_layer_list(dr):
    """Section 3.1's approximate stem: pool strides multiplied into conv1 / conv2, LRN pruned; the rest as DR_ARCH_GOOGLENET."""
    net = dr.Net(dr.DR_ARCH_GOOGLENET_STREAMLINE, dr.DR_MODE_SLIM, 1)
    ref = dr.Net(dr.DR_ARCH_GOOGLENET, dr.DR_MODE_SLIM, 1)
    assert net.dr_net_num_layers() == ref.dr_net_num_layers() + 1       # + the space-to-depth copy in front of conv1
    infos = {net.dr_net_layer_info(i)["name"]: net.dr_net_layer_info(i) for i in range(net.dr_net_num_layers())}
    rinfos = {ref.dr_net_layer_info(i)["name"]: ref.dr_net_layer_info(i) for i in range(ref.dr_net_num_layers())}
    assert infos["conv1"]["dims"] == (1, 56, 56, 64) and infos["conv2"]["dims"] == (1, 28, 28, 192)
    # stride 4 instead of 2: a quarter of conv1's multiply-adds; stride 2 instead of 1: a quarter of conv2's
    assert abs(infos["conv1"]["flops"] * 4 - rinfos["conv1"]["flops"]) <= 1e-6 * rinfos["conv1"]["flops"]
    assert abs(infos["conv2"]["flops"] * 4 - rinfos["conv2"]["flops"]) <= 1e-6 * rinfos["conv2"]["flops"]
    assert infos["3a.m5"]["dims"] == rinfos["3a.m5"]["dims"] and infos["fc"]["dims"] == rinfos["fc"]["dims"]
    uns = dr.Net(dr.DR_ARCH_GOOGLENET_STREAMLINE, dr.DR_MODE_UNSLIMMED, 1)
    names = [uns.dr_net_layer_info(i)["name"] for i in range(uns.dr_net_num_layers())]
    assert "conv1.pool" not in names and "conv2.lrn" not in names and "conv1.conv" in names
    assert infos["conv1.s2d"]["kind"] == 1 and infos["conv1.s2d"]["dims"] == (1, 57, 57, 64)   # 7x7/4 -> 2x2/1 over 64 channels


def test_alexnet_layer_list(dr):
    """AlexNet (Section 4.3): conv1 + norm1 and conv2 + norm2 as slim layers; 227x227 input only."""
    net = dr.Net(dr.DR_ARCH_ALEXNET, dr.DR_MODE_SLIM, 2, 227, 227)
    infos = [net.dr_net_layer_info(i) for i in range(net.dr_net_num_layers())]
    assert [i["name"] for i in infos] == ["conv1.s2d", "conv1", "pool1", "conv2", "pool2", "conv3", "conv4", "conv5", "pool5", "fc6", "fc7", "fc8"]
    li = {i["name"]: i for i in infos}
    assert li["conv1.s2d"]["dims"] == (2, 57, 57, 64) and li["conv1"]["dims"] == (2, 55, 55, 96) and li["pool1"]["dims"] == (2, 27, 27, 96)
    assert li["conv2"]["dims"] == (2, 27, 27, 256) and li["pool5"]["dims"] == (2, 6, 6, 256) and li["fc8"]["dims"] == (2, 1, 1, 1000)
    assert li["conv1"]["flops"] == 2.0 * 2 * 55 * 55 * 96 * 11 * 11 * 3           # of the 11x11/4 layer, not of its re-laid form
    assert li["conv2"]["flops"] == 2.0 * 2 * 27 * 27 * 256 * 25 * 48              # grouped: half of the dense stand-in
    names = [net.dr_net_param_spec(i)[0] for i in range(net.dr_net_num_params())]
    assert net.dr_net_param_spec(names.index("conv2.w"))[1] == (256, 5, 5, 48)
    with pytest.raises(dr.DrError) as e:
        dr.Net(dr.DR_ARCH_ALEXNET, dr.DR_MODE_SLIM, 1, 224, 224)
    assert e.value.status == dr.DR_ERR_INVALID_ARG


def test_resnet50_layer_lists(dr):
    slim = dr.Net(dr.DR_ARCH_RESNET50, dr.DR_MODE_SLIM, 1)
    n = slim.dr_net_num_layers()
    infos = [slim.dr_net_layer_info(i) for i in range(n)]
    assert sum(i["kind"] == 0 for i in infos) == 54 and n == 55      # 53 convs + fc, + avg-pool
    total = sum(i["flops"] for i in infos)
    assert abs(total / 1e9 - 7.72) < 0.02
    names = {i["name"]: i for i in infos}
    assert names["res3a.2a"]["dims"] == (1, 28, 28, 128)             # stride 2 on the first 1x1
    assert names["res5c.2c"]["dims"] == (1, 7, 7, 2048)
    uns = dr.Net(dr.DR_ARCH_RESNET50, dr.DR_MODE_UNSLIMMED, 1)
    ku = [uns.dr_net_layer_info(i) for i in range(uns.dr_net_num_layers())]
    assert sum(i["kind"] == 0 for i in ku) == 54
    # every conv is followed by BatchNorm and Scale launches of their own
    assert sum(i["name"].endswith(".bn") for i in ku) == 53
    with pytest.raises(dr.DrError):
        dr.Net(7, 0, 1)
    with pytest.raises(dr.DrError):
        dr.Net(0, 0, 1, 16, 16)


def header_defines():
    """{name: integer value} of the plain integer #defines of include/dr.h."""
    text = open(os.path.join(ROOT, "include", "dr.h")).read()
    out = {}
    for name, val in re.findall(r"^#define[ \t]+(DR_[A-Z0-9_]+)[ \t]+([^/\n]+)", text, flags=re.M):
        expr = re.sub(r"(?<=[0-9a-fA-F])[uU]\b", "", val.strip())
        if re.fullmatch(r"[-()0-9a-fA-FxX<\s]+", expr):
            out[name] = int(eval(expr, {"__builtins__": {}}))
    return out


def test_python_constants_mirror_the_header(dr):
    """Every integer constant the binding repeats has the header's value (flags, codes, kernel paths, sizes)."""
    defs = header_defines()
    assert defs["DR_INCEPTION_STATIC_SCRATCH_BYTES"] == 4 << 20
    checked = 0
    for name, val in defs.items():
        if hasattr(dr, name):
            assert getattr(dr, name) == val, (name, getattr(dr, name), val)
            checked += 1
    assert checked >= 30
    for need in ("DR_INCEPTION_STATIC_SCRATCH_BYTES", "DR_CONV_WS_COUNTER_BYTES", "DR_PATH_UMMA_QLIN", "DR_ERR_DEVICE_TIMEOUT", "DR_OUT_F32"):
        assert need in defs and hasattr(dr, need), need
    assert set(dr.PATH_NAMES) == {-1} | {v for k, v in defs.items() if k.startswith("DR_PATH_")}


def test_conv_plan_is_host_only_and_names_the_kernel(dr):
    n0 = dr.dr_launch_count()
    big = dr.dr_conv_plan(dr.dr_conv_desc(k=5, stride=1, pad=2, Cin=528, Cout=512, flags=dr.DR_BIAS | dr.DR_RELU), 256, 14, 14)
    assert big["path"] == "umma_tma" and big["pair"] == 1 and big["Nt"] * big["n_blocks"] * (2 if big["wide"] else 1) >= 512
    stem = dr.dr_conv_plan(dr.dr_conv_desc(k=7, stride=2, pad=3, Cin=3, Cout=64, flags=dr.DR_BIAS | dr.DR_RELU | dr.DR_POOL | dr.DR_LRN,
                                           pool_k=3, pool_stride=2, pool_pad=1, lrn_size=5, lrn_alpha=1e-4, lrn_beta=0.75, lrn_k=1.0), 1, 64, 64)
    assert stem["path"].startswith("umma_stem")
    d = dr.dr_conv_desc(k=5, stride=1, pad=2, Cin=832, Cout=640, flags=dr.DR_BIAS | dr.DR_RELU)
    assert dr.dr_conv_plan(d, 1, 7, 7, dr.dr_conv_workspace_bytes(d, 1, 7, 7))["path"] == "umma_splitk"
    assert dr.dr_conv_plan(d, 1, 7, 7, 0)["path"] != "umma_splitk"
    with pytest.raises(dr.DrError) as e:
        dr.dr_conv_plan(dr.dr_conv_desc(k=0, stride=1, pad=0, Cin=8, Cout=8, flags=0), 1, 8, 8)
    assert e.value.status == dr.DR_ERR_INVALID_ARG
    assert dr.dr_launch_count() == n0
