"""Whole-network GPU parity: slimmed GoogLeNet (batch 1 and 256) and ResNet-50 (batch 128).

Per-layer checks are teacher-forced: the CPU checker's layer l is fed what the GPU stored for
layer l-1, so each figure measures one layer.  Logits are compared free-running.  At the large
batches the checker runs a seeded subset of the batch entries (each image is independent through
every layer), with full per-layer outputs for entry 0.
"""
import numpy as np
import pytest

import dr_synth as S
import dr_synth.params as P
from util import LOGITS_L2, assert_layer_close, err_norms, load_params, to_dev_bf16, to_host, _wrap

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dr():
    import paper_1708_04728_b200 as dr
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    return dr


def run_net(dr, arch, mode, B, params, x_entries_fn, hw=224):
    """Build, prepare and run a net on the seeded batch; returns (net, workspace, logits, keepalive)."""
    import torch
    net = dr.Net(arch, mode, B, hw, hw)
    keep = []
    load_params(net, params, keep)
    ws = torch.empty(net.dr_net_workspace_bytes() + 256, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 256
    ws = ws[off:]
    x = torch.empty((B, hw, hw, 3), dtype=torch.bfloat16, device="cuda")
    step = 16
    for n0 in range(0, B, step):
        x[n0:n0 + step] = to_dev_bf16(x_entries_fn(range(n0, min(B, n0 + step))))
    logits = torch.full((B, 1000), float("nan"), dtype=torch.float32, device="cuda")
    net.dr_net_prepare(ws)
    net.dr_net_forward(x, ws, logits)
    st, info = dr.dr_device_status()
    assert st == 0, f"device status {st} {info}"
    keep += [ws, x]
    return net, ws, logits, keep


def layer_outputs(net, logits, entries):
    """{layer name: float64 [len(entries),H,W,C]} of the slices the layers wrote, for some batch entries."""
    import torch
    out = {}
    idx = torch.as_tensor(list(entries), device="cuda")
    for i in range(net.dr_net_num_layers()):
        li = net.dr_net_layer_info(i)
        B, H, W, Cc = li["dims"]
        if li["is_f32"]:
            out[li["name"]] = to_host(logits[idx]).reshape(len(entries), 1, 1, Cc)
            continue
        n_el = (B * H * W - 1) * li["ldc"] + Cc
        t = torch.as_strided(_wrap(li["ptr"], n_el), (B, H, W, Cc), (H * W * li["ldc"], W * li["ldc"], li["ldc"], 1))
        out[li["name"]] = to_host(t[idx])
    return out


def check_network(dr, arch, B, entries, steps_fn, params, per_layer_tol=None, hw=224, out="fc"):
    import oracle.nets as N
    images = lambda rng: np.stack([S.normal(0, f"x[{n}]", (hw, hw, 3)) for n in rng])
    net, ws, logits, keep = run_net(dr, arch, dr.DR_MODE_SLIM, B, params, images, hw=hw)
    paths = {net.dr_net_layer_info(i)["name"]: net.dr_net_layer_info(i)["conv_path"] for i in range(net.dr_net_num_layers())}
    steps = steps_fn(params)
    # ---- per layer, teacher-forced: batch entry 0 and, at batch > 1, the last entry (where the ragged last tile, the odd
    # tile of a CTA pair and the tail of the per-stream ranges live at full size); logits for all checked entries
    report = []
    for e in ([entries[0]] + ([B - 1] if B > 1 else [])):
        G = layer_outputs(net, logits, [e])
        x0 = images([e])
        if arch == dr.DR_ARCH_GOOGLENET_PAPER:
            # reducers are stored in tensors rounded up to 64 channels: the extra channels must be exactly zero
            widths = {k: v.shape[-1] for k, v in N.run(steps, x0).items()}
            for name, c in widths.items():
                if name in G and G[name].shape[-1] > c:
                    assert not np.any(G[name][..., c:]), f"{name}: padded channels are not zero"
                    G[name] = G[name][..., :c]
        given = dict(G)
        for st in steps:                      # concatenated module outputs are re-assembled from their slices
            if st.virtual:
                given[st.name] = np.concatenate([given[s] for s in st.src], axis=-1)
        forced = N.run(steps, x0, given=given)
        for st in steps:
            if st.virtual:
                continue
            assert st.name in G, f"GPU net has no layer {st.name}"
            mx, l2 = assert_layer_close(G[st.name], forced[st.name], f"{st.name} (batch entry {e})")
            report.append((st.name, paths.get(st.name), mx, l2))
    # ---- end to end, free-running, the seeded subset
    xs = images(entries)
    free = N.run(steps, xs)
    got = to_host(logits[list(entries)]).reshape(len(entries), 1, 1, 1000)
    assert np.all(np.isfinite(got))
    for i in range(len(entries)):
        mx, l2 = err_norms(got[i], free[out][i])
        assert l2 <= LOGITS_L2, f"logits of batch entry {entries[i]}: rel-L2 {l2:.3e} > {LOGITS_L2}"
    # every batch entry produced something finite
    assert bool(np.isfinite(to_host(logits)).all())
    worst = max(report, key=lambda r: r[3])
    print(f"\n[{['googlenet','resnet50','googlenet-paper','googlenet-streamline','alexnet'][arch]} B={B}] worst layer {worst[0]} path={worst[1]} max {worst[2]:.2e} l2 {worst[3]:.2e}; "
          f"logits rel-L2 {max(err_norms(got[i], free[out][i])[1] for i in range(len(entries))):.2e}")
    return net, logits, free, keep


def subset(B, k):
    """Entry 0, the last entry (B - 1), then the first entries of a seeded permutation."""
    fixed = [0] + ([B - 1] if B > 1 and k > 1 else [])
    rest = [int(i) for i in S.stream(0, "subset").permutation(B) if i not in fixed]
    return (fixed + rest)[:max(k, 1)]


@pytest.mark.parametrize("B,k", [(1, 1), (256, 4)])
def test_googlenet_slim(dr, B, k):
    import oracle.nets as N
    params = P.googlenet_params(0)
    check_network(dr, dr.DR_ARCH_GOOGLENET, B, subset(B, k), N.googlenet_steps, params)


@pytest.mark.parametrize("B,k", [(1, 1), (64, 2)])
def test_googlenet_paper_form(dr, B, k):
    """GoogLeNet slimmed the paper's own way (two branches per module): per-layer and logits parity."""
    import oracle.nets as N
    params = P.googlenet_paper_params(0)
    check_network(dr, dr.DR_ARCH_GOOGLENET_PAPER, B, subset(B, k), N.googlenet_paper_steps, params)


@pytest.mark.parametrize("B,k", [(1, 1), (64, 2)])
def test_googlenet_streamline_form(dr, B, k):
    """GoogLeNet with the stem in Section 3.1's approximate form (7x7/4, 3x3/2, no pool, no LRN): parity with its own definition."""
    import oracle.nets as N
    params = P.googlenet_params(0)
    check_network(dr, dr.DR_ARCH_GOOGLENET_STREAMLINE, B, subset(B, k), N.googlenet_streamline_steps, params)


@pytest.mark.parametrize("B,k", [(1, 1), (32, 2)])
def test_alexnet_slim(dr, B, k):
    """AlexNet with conv1 + norm1 and conv2 + norm2 as slim layers (Section 4.3), grouped layers as block-diagonal
    dense convolutions: per-layer and logits parity with the grouped, unfused checker."""
    import oracle.nets as N
    params = P.alexnet_params(0)
    net, logits, free, keep = check_network(dr, dr.DR_ARCH_ALEXNET, B, subset(B, k), N.alexnet_steps, params, hw=227, out="fc8")
    names = [net.dr_net_layer_info(i)["name"] for i in range(net.dr_net_num_layers())]
    assert names == ["conv1.s2d", "conv1", "pool1", "conv2", "pool2", "conv3", "conv4", "conv5", "pool5", "fc6", "fc7", "fc8"]
    # the baseline runs ReLU and LRN as layers of their own
    uns = dr.Net(dr.DR_ARCH_ALEXNET, dr.DR_MODE_UNSLIMMED, B, 227, 227)
    assert uns.dr_net_num_layers() == 12 + 7 + 2


@pytest.mark.parametrize("B,k", [(128, 2)])
def test_resnet50_slim(dr, B, k):
    import oracle.nets as N
    params = P.resnet50_params(0)
    check_network(dr, dr.DR_ARCH_RESNET50, B, subset(B, k), N.resnet50_steps, params)


@pytest.mark.parametrize("arch", [0, 1, 2])
def test_unslimmed_path_matches(dr, arch):
    """The layer-by-layer baseline computes the same function: logits vs the checker and vs the slim net."""
    import oracle.nets as N
    B = 2
    params = [P.googlenet_params, P.resnet50_params, P.googlenet_paper_params][arch](0)
    steps = [N.googlenet_steps, N.resnet50_steps, N.googlenet_paper_steps][arch](params)
    images = lambda rng: np.stack([S.normal(0, f"x[{n}]", (224, 224, 3)) for n in rng])
    net_u, _, logits_u, keep_u = run_net(dr, arch, dr.DR_MODE_UNSLIMMED, B, params, images)
    net_s, _, logits_s, keep_s = run_net(dr, arch, dr.DR_MODE_SLIM, B, params, images)
    free = N.run(steps, images(range(B)))
    gu, gs = to_host(logits_u), to_host(logits_s)
    for i in range(B):
        assert err_norms(gu[i], free["fc"][i].reshape(-1))[1] <= LOGITS_L2
        assert err_norms(gs[i], free["fc"][i].reshape(-1))[1] <= LOGITS_L2
        assert err_norms(gu[i], gs[i])[1] <= LOGITS_L2
    # the baseline launches every non-tensor layer separately
    n_u = sum(net_u.dr_net_layer_info(i)["kind"] == 1 for i in range(net_u.dr_net_num_layers()))
    n_s = sum(net_s.dr_net_layer_info(i)["kind"] == 1 for i in range(net_s.dr_net_num_layers()))
    assert n_u > 10 * n_s
    # group outputs of the baseline (several bf16 roundings inside one group) stay close to the checker's
    G = layer_outputs(net_u, logits_u, [0])
    for name in ("conv1", "conv2", "3a", "5b") if arch != 1 else ("conv1", "res2a.2c", "res5c.2c"):
        if name in G:
            mx, l2 = err_norms(G[name], free[name][:1])
            assert l2 <= 2e-2, (name, l2)


def test_net_timing_and_launch_count(dr):
    params = P.googlenet_params(0)
    images = lambda rng: np.stack([S.normal(0, f"x[{n}]", (224, 224, 3)) for n in rng])
    net, ws, logits, keep = run_net(dr, dr.DR_ARCH_GOOGLENET, dr.DR_MODE_SLIM, 1, params, images)
    x = keep[-1]
    n0 = dr.dr_launch_count()
    net.dr_net_set_timing(True)
    net.dr_net_forward(x, ws, logits)
    assert dr.dr_launch_count() - n0 == net.dr_net_num_layers()
    total = sum(net.dr_net_layer_time_us(i) for i in range(net.dr_net_num_layers()))
    assert total > 0
    first = to_host(logits).copy()
    net.dr_net_forward(x, ws, logits)                  # deterministic: no atomics anywhere
    assert np.array_equal(first, to_host(logits))
    # tensor maps are remembered by what they were encoded from: further passes over the same buffers encode none
    net.dr_net_set_timing(False)
    net.dr_net_forward(x, ws, logits)                  # (layers that share a launch sum in another order than when timed apart)
    untimed = to_host(logits).copy()
    e0 = dr.dr_tensor_map_encodes()
    assert e0 > 0
    net.dr_net_forward(x, ws, logits)
    net.dr_net_forward(x, ws, logits)
    assert dr.dr_tensor_map_encodes() == e0
    assert np.array_equal(untimed, to_host(logits))


@pytest.mark.parametrize("env", [{"DR_SPLITK_CLUSTER": "1"}, {"DR_SPLITK_CLUSTER": "1", "DR_SPLITK_OWN_CTAS": "0"}, {"DR_SPLITK_CLUSTER": "8"},
                                 {"DR_NET_PDL": "0"}])
def test_single_image_forward_in_the_other_hand_over_forms(env):
    """The split-K launch of an inception module has several forms chosen per process (hand-over through L2 or through a
    cluster's shared memory, the 3x3 on CTAs of its own or behind the reducer, programmatic launches or ordinary ones): the
    single-image network passes its parity test in each of them."""
    import os
    import subprocess
    import sys
    e = dict(os.environ)
    e.update(env)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_net.py"), "-q", "-x", "-m", "gpu", "-k", "test_googlenet_slim and 1-1",
                        "-p", "no:cacheprovider"], cwd=root, env=e, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert "1 passed" in r.stdout, r.stdout[-2000:]
