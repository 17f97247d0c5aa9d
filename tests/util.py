"""Helpers for the GPU parity tests: host<->device movement and error norms (no method arithmetic)."""
import numpy as np


def gpu_available():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def to_dev_bf16(a):
    """float32 numpy array holding bfloat16-representable values -> cuda bfloat16 tensor (exact)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(torch.bfloat16)
    return t


def to_dev_f32(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def to_host(t):
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def err_norms(got, ref):
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0, 0.0
    d = got - ref
    mx = float(np.abs(d).max() / max(np.abs(ref).max(), 1e-30))
    l2 = float(np.sqrt((d * d).sum()) / max(np.sqrt((ref * ref).sum()), 1e-30))
    return mx, l2


# the per-layer bar: max|err| <= 1e-2 * max|ref| and relative L2 <= 4e-3
LAYER_MAX, LAYER_L2, LOGITS_L2 = 1e-2, 4e-3, 2e-2


def assert_layer_close(got, ref, what=""):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    mx, l2 = err_norms(got, ref)
    assert mx <= LAYER_MAX and l2 <= LAYER_L2, f"{what}: max-rel {mx:.3e} (<= {LAYER_MAX}), rel-L2 {l2:.3e} (<= {LAYER_L2})"
    return mx, l2


def load_params(net, params, keep):
    """Upload a name->array dict into a Net by its parameter specs; `keep` collects the tensors."""
    for i in range(net.dr_net_num_params()):
        name, dims, is_f32, count = net.dr_net_param_spec(i)
        a = params[name]
        assert a.size == count, (name, a.shape, dims)
        t = to_dev_f32(a) if is_f32 else to_dev_bf16(a)
        keep.append(t)
        net.dr_net_set_param(i, t)


def net_layer_outputs(net, logits):
    """{layer name: float64 array of the slice that layer wrote}, read back from the workspace."""
    import ctypes
    import torch
    out = {}
    for i in range(net.dr_net_num_layers()):
        li = net.dr_net_layer_info(i)
        B, H, W, Cc = li["dims"]
        if li["name"] == "fc":
            out["fc"] = to_host(logits).reshape(B, 1, 1, Cc)
            continue
        # view of the strided slice through a uint8 tensor aliasing the workspace is overkill:
        # copy rows with cudaMemcpy2D semantics via torch.as_strided on a wrapped pointer
        n_el = (B * H * W - 1) * li["ldc"] + Cc
        buf = _wrap(li["ptr"], n_el)
        t = torch.as_strided(buf, (B, H, W, Cc), (H * W * li["ldc"], W * li["ldc"], li["ldc"], 1))
        out[li["name"]] = to_host(t)
    return out


def _wrap(ptr, n_el):
    """bfloat16 torch view of raw device memory (no copy, no ownership)."""
    import torch

    class _Holder:
        pass
    h = _Holder()
    h.__cuda_array_interface__ = {"shape": (n_el,), "typestr": "<i2", "data": (int(ptr), False), "version": 2}
    return torch.as_tensor(h, device="cuda").view(torch.bfloat16)
