"""Python binding of libdeeprebirth (argument marshalling only).

Every function has the name and argument order of its C entry point in ``include/dr.h``;
tensors may be passed as ``torch.Tensor`` (their ``data_ptr()`` is taken) or as integer device
addresses, streams as ``torch.cuda.Stream``, an integer handle, or ``None`` (the current torch
stream).  All arithmetic happens in the CUDA library; importing this module without the built
library raises.  A non-zero status raises ``DrError``.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdeeprebirth.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python paper_1708_04728_b200/build.py` "
        "(there is no CPU or PyTorch fallback)")

_lib = C.CDLL(LIB_PATH)

# status codes / flags (mirrors of include/dr.h)
DR_OK, DR_ERR_INVALID_ARG, DR_ERR_UNSUPPORTED, DR_ERR_ALIGNMENT = 0, -1, -2, -3
DR_ERR_WORKSPACE, DR_ERR_CUDA, DR_ERR_DEVICE_TIMEOUT = -4, -5, -6
DR_BIAS, DR_RELU, DR_POOL, DR_LRN, DR_RESIDUAL = 0x01, 0x02, 0x04, 0x08, 0x10
DR_LRN_BEFORE_POOL, DR_RELU_AFTER_RESIDUAL, DR_OUT_F32 = 0x20, 0x40, 0x80
DR_ARCH_GOOGLENET, DR_ARCH_RESNET50, DR_ARCH_GOOGLENET_PAPER, DR_ARCH_GOOGLENET_STREAMLINE, DR_ARCH_ALEXNET = 0, 1, 2, 3, 4
DR_MODE_SLIM, DR_MODE_UNSLIMMED = 0, 1
DR_PATH_AUTO, DR_PATH_SIMT, DR_PATH_UMMA_GATHER, DR_PATH_UMMA_TMA, DR_PATH_UMMA_PATCH, DR_PATH_UMMA_STEM, DR_PATH_RETIRED_6, DR_PATH_UMMA_STEM_D = 0, 1, 2, 3, 4, 5, 6, 7
DR_PATH_UMMA_SPLITK = 8
DR_PATH_UMMA_QLIN = 9
DR_CONV_WS_COUNTER_BYTES = 1024
PATH_NAMES = {0: "auto", 1: "simt", 2: "umma_gather", 3: "umma_tma", 4: "umma_patch", 5: "umma_stem", 6: "retired", 7: "umma_stem_d",
              8: "umma_splitk", 9: "umma_qlin", -1: "-"}


class dr_conv_desc(C.Structure):
    _fields_ = [("k", C.c_int), ("stride", C.c_int), ("pad", C.c_int), ("Cin", C.c_int), ("Cout", C.c_int),
                ("flags", C.c_uint), ("pool_k", C.c_int), ("pool_stride", C.c_int), ("pool_pad", C.c_int),
                ("lrn_size", C.c_int), ("lrn_alpha", C.c_float), ("lrn_beta", C.c_float), ("lrn_k", C.c_float),
                ("y_ldc", C.c_int), ("y_coff", C.c_int)]


class dr_inception_desc(C.Structure):
    _fields_ = [("Cin", C.c_int), ("c3r", C.c_int), ("c3", C.c_int), ("cm", C.c_int), ("pool_after", C.c_int)]


class dr_param_spec(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("dims", C.c_int * 4), ("is_f32", C.c_int), ("count", C.c_size_t)]


class dr_layer_info(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("kind", C.c_int), ("dims", C.c_int * 4), ("ldc", C.c_int),
                ("coff", C.c_int), ("is_f32", C.c_int), ("ptr", C.c_void_p), ("flops", C.c_double),
                ("bytes", C.c_double), ("conv_path", C.c_int)]


class DrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {dr_strerror(status)} ({status})")


_P, _I, _F, _Z = C.c_void_p, C.c_int, C.c_float, C.c_size_t
_SIGS = {
    "dr_strerror": (C.c_char_p, [_I]),
    "dr_fold_bn": (_I, [_I, _I, _P, _P, _P, _P, _F, _F, _P, _P, _P, _P, _P]),
    "dr_embed_filter": (_I, [_I, _I, _I, _I, _P, _I, _P, _P]),
    "dr_embed_groups": (_I, [_I, _I, _I, _I, _P, _P, _P]),
    "dr_space_to_depth": (_I, [_I, _I, _I, _I, _I, _I, _I, _I, _P, _P, _P]),
    "dr_s2d_filter": (_I, [_I, _I, _I, _I, _I, _P, _P, _P]),
    "dr_s2d_filter_grad": (_I, [_I, _I, _I, _I, _I, _P, _P, _P]),
    "dr_conv_slim": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, _P, _P, _P, _P, _P, _P, _P]),
    "dr_regress_workspace_bytes": (_I, [_I, C.POINTER(_Z)]),
    "dr_regress_grad": (_I, [_I, _I, _I, _I, _P, _P, _I, _P, _P, _P, _P, _Z, _P]),
    "dr_regress_grad_shard": (_I, [_I, _I, _I, _I, _I, _P, _P, _I, _P, _P, _P, _P, _Z, _P]),
    "dr_regress_shard_grads": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, _I, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _Z, _P]),
    "dr_conv_wgrad_workspace_bytes": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, C.POINTER(_Z)]),
    "dr_conv_wgrad": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, _P, _P, _P, _P, _Z, _P]),
    "dr_sgd_update": (_I, [_Z, _P, _P, _P, _F, _F, _F, _P, _P]),
    "dr_regress_step_workspace_bytes": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, C.POINTER(_Z)]),
    "dr_regress_step": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, _P, _P, _P, _P, _P, _P, _P, _F, _F, _F, _P, _P, _P, _P, _P, _P, _Z, _P]),
    "dr_conv_workspace_bytes": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, C.POINTER(_Z)]),
    "dr_conv_slim_ws": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, _P, _P, _P, _P, _P, _P, _P, _Z, _P]),
    "dr_inception_workspace_bytes": (_I, [C.POINTER(dr_inception_desc), _I, _I, _I, C.POINTER(_Z)]),
    "dr_inception_slim": (_I, [C.POINTER(dr_inception_desc), _I, _I, _I, _P, C.POINTER(_P), C.POINTER(_P), _P, _P, _P]),
    "dr_inception_slim_static": (_I, [C.POINTER(dr_inception_desc), _I, _I, _I, _P, C.POINTER(_P), C.POINTER(_P), _P, _P]),
    "dr_relu": (_I, [_Z, _P, _P, _P]),
    "dr_maxpool": (_I, [_I, _I, _I, _I, _I, _I, _I, _P, _P, _P, _P]),
    "dr_lrn": (_I, [_I, _I, _I, _I, _I, _F, _F, _F, _P, _P, _P]),
    "dr_bn": (_I, [_I, _I, _I, _I, _P, _P, _P, _F, _F, _P, _P, _P, _P]),
    "dr_scale": (_I, [_I, _I, _I, _I, _P, _P, _P, _P, _P]),
    "dr_add": (_I, [_Z, _P, _P, _P, _P]),
    "dr_concat": (_I, [_Z, _I, _P, _I, _I, _P, _P]),
    "dr_avgpool_global": (_I, [_I, _I, _I, _I, _P, _P, _P]),
    "dr_net_create": (_I, [C.POINTER(_P), _I, _I, _I, _I, _I]),
    "dr_net_destroy": (_I, [_P]),
    "dr_net_num_params": (_I, [_P]),
    "dr_net_param_spec": (_I, [_P, _I, C.POINTER(dr_param_spec)]),
    "dr_net_set_param": (_I, [_P, _I, _P]),
    "dr_net_workspace_bytes": (_I, [_P, C.POINTER(_Z)]),
    "dr_net_prepare": (_I, [_P, _P, _P]),
    "dr_net_forward": (_I, [_P, _P, _P, _P, _P]),
    "dr_net_num_layers": (_I, [_P]),
    "dr_net_layer_info": (_I, [_P, _I, C.POINTER(dr_layer_info)]),
    "dr_net_set_timing": (_I, [_P, _I]),
    "dr_net_layer_time_us": (_I, [_P, _I, C.POINTER(_F)]),
    "dr_net_activation_bytes": (_I, [_P, C.POINTER(_Z)]),
    "dr_set_conv_path": (_I, [_I]),
    "dr_last_conv_path": (_I, []),
    "dr_device_status": (_I, [C.POINTER(_I)]),
    "dr_selftest_wait_timeout": (_I, [C.c_longlong, _P]),
    "dr_launch_count": (C.c_longlong, []),
    "dr_tensor_map_encodes": (C.c_longlong, []),
    "dr_conv_plan": (_I, [C.POINTER(dr_conv_desc), _I, _I, _I, _Z, C.POINTER(_I)]),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(_lib, _name)          # AttributeError here = the library does not export it
    _fn.restype, _fn.argtypes = _res, _args

EXPORTS = tuple(_SIGS)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(s):
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _check(status: int, where: str):
    if status != DR_OK:
        raise DrError(status, where)


def dr_strerror(status: int) -> str:
    return _lib.dr_strerror(status).decode()


def dr_fold_bn(Cout, K, w_in, b_in, mean, var, m, eps, gamma, beta, w_out, b_out, stream=None):
    _check(_lib.dr_fold_bn(Cout, K, _ptr(w_in), _ptr(b_in), _ptr(mean), _ptr(var), m, eps, _ptr(gamma), _ptr(beta),
                           _ptr(w_out), _ptr(b_out), _stream(stream)), "dr_fold_bn")


def dr_embed_filter(Cout, Cin, ks, kb, w_small, joff, w_big, stream=None):
    _check(_lib.dr_embed_filter(Cout, Cin, ks, kb, _ptr(w_small), joff, _ptr(w_big), _stream(stream)), "dr_embed_filter")


def dr_embed_groups(Cout, Cin_g, k, groups, w_grouped, w_dense, stream=None):
    _check(_lib.dr_embed_groups(Cout, Cin_g, k, groups, _ptr(w_grouped), _ptr(w_dense), _stream(stream)), "dr_embed_groups")


def dr_space_to_depth(B, H, W, Cc, k, s, pad, Cp, x, y, stream=None):
    _check(_lib.dr_space_to_depth(B, H, W, Cc, k, s, pad, Cp, _ptr(x), _ptr(y), _stream(stream)), "dr_space_to_depth")


def dr_s2d_filter(Cout, k, Cc, s, Cp, w, w_out, stream=None):
    _check(_lib.dr_s2d_filter(Cout, k, Cc, s, Cp, _ptr(w), _ptr(w_out), _stream(stream)), "dr_s2d_filter")


def dr_s2d_filter_grad(Cout, k, Cc, s, Cp, dw_s2d, dw, stream=None):
    _check(_lib.dr_s2d_filter_grad(Cout, k, Cc, s, Cp, _ptr(dw_s2d), _ptr(dw), _stream(stream)), "dr_s2d_filter_grad")


def dr_conv_slim(desc, B, H, W, x, w, b, residual, y, argmax=None, stream=None):
    _check(_lib.dr_conv_slim(C.byref(desc), B, H, W, _ptr(x), _ptr(w), _ptr(b), _ptr(residual), _ptr(y), _ptr(argmax),
                             _stream(stream)), "dr_conv_slim")


def dr_regress_workspace_bytes(Cc) -> int:
    n = _Z(0)
    _check(_lib.dr_regress_workspace_bytes(Cc, C.byref(n)), "dr_regress_workspace_bytes")
    return n.value


def dr_regress_grad(B, H, W, Cc, y, yt, relu, dz, db, loss, workspace, workspace_bytes, stream=None):
    _check(_lib.dr_regress_grad(B, H, W, Cc, _ptr(y), _ptr(yt), int(relu), _ptr(dz), _ptr(db), _ptr(loss), _ptr(workspace),
                                workspace_bytes, _stream(stream)), "dr_regress_grad")


def dr_conv_wgrad_workspace_bytes(desc, B, H, W) -> int:
    n = _Z(0)
    _check(_lib.dr_conv_wgrad_workspace_bytes(C.byref(desc), B, H, W, C.byref(n)), "dr_conv_wgrad_workspace_bytes")
    return n.value


def dr_conv_wgrad(desc, B, H, W, x, dz, dw, workspace, workspace_bytes, stream=None):
    _check(_lib.dr_conv_wgrad(C.byref(desc), B, H, W, _ptr(x), _ptr(dz), _ptr(dw), _ptr(workspace), workspace_bytes,
                              _stream(stream)), "dr_conv_wgrad")


def dr_sgd_update(n, w, v, g, lr, momentum, decay, w_bf16=None, stream=None):
    _check(_lib.dr_sgd_update(n, _ptr(w), _ptr(v), _ptr(g), lr, momentum, decay, _ptr(w_bf16), _stream(stream)), "dr_sgd_update")


def dr_regress_step_workspace_bytes(desc, B, H, W) -> int:
    n = _Z(0)
    _check(_lib.dr_regress_step_workspace_bytes(C.byref(desc), B, H, W, C.byref(n)), "dr_regress_step_workspace_bytes")
    return n.value


def dr_regress_step(desc, B, H, W, x, yt, w, b, vw, vb, w_bf16, lr, momentum, decay, y, dz, dw, db, loss, workspace,
                    workspace_bytes, stream=None):
    _check(_lib.dr_regress_step(C.byref(desc), B, H, W, _ptr(x), _ptr(yt), _ptr(w), _ptr(b), _ptr(vw), _ptr(vb), _ptr(w_bf16),
                                lr, momentum, decay, _ptr(y), _ptr(dz), _ptr(dw), _ptr(db), _ptr(loss), _ptr(workspace),
                                workspace_bytes, _stream(stream)), "dr_regress_step")


def dr_regress_grad_shard(B, batch, H, W, Cc, y, yt, relu, dz, db, loss, workspace, workspace_bytes, stream=None):
    _check(_lib.dr_regress_grad_shard(B, batch, H, W, Cc, _ptr(y), _ptr(yt), int(relu), _ptr(dz), _ptr(db), _ptr(loss), _ptr(workspace),
                                      workspace_bytes, _stream(stream)), "dr_regress_grad_shard")


def dr_regress_shard_grads(desc, B, batch, H, W, x, yt, w_bf16, b, y, dz, dw, db, loss, workspace, workspace_bytes, stream=None):
    _check(_lib.dr_regress_shard_grads(C.byref(desc), B, batch, H, W, _ptr(x), _ptr(yt), _ptr(w_bf16), _ptr(b), _ptr(y), _ptr(dz), _ptr(dw),
                                       _ptr(db), _ptr(loss), _ptr(workspace), workspace_bytes, _stream(stream)), "dr_regress_shard_grads")


def dr_conv_workspace_bytes(desc, B, H, W) -> int:
    n = _Z(0)
    _check(_lib.dr_conv_workspace_bytes(C.byref(desc), B, H, W, C.byref(n)), "dr_conv_workspace_bytes")
    return n.value


def dr_conv_slim_ws(desc, B, H, W, x, w, b, residual, y, argmax, workspace, workspace_bytes, stream=None):
    _check(_lib.dr_conv_slim_ws(C.byref(desc), B, H, W, _ptr(x), _ptr(w), _ptr(b), _ptr(residual), _ptr(y), _ptr(argmax),
                                _ptr(workspace), workspace_bytes, _stream(stream)), "dr_conv_slim_ws")


def dr_inception_workspace_bytes(desc, B, H, W) -> int:
    n = _Z(0)
    _check(_lib.dr_inception_workspace_bytes(C.byref(desc), B, H, W, C.byref(n)), "dr_inception_workspace_bytes")
    return n.value


def dr_inception_slim(desc, B, H, W, x, w, b, y, workspace, stream=None):
    wa = (_P * 3)(*[_ptr(t) for t in w])
    ba = (_P * 3)(*[_ptr(t) for t in b])
    _check(_lib.dr_inception_slim(C.byref(desc), B, H, W, _ptr(x), wa, ba, _ptr(y), _ptr(workspace), _stream(stream)),
           "dr_inception_slim")


DR_INCEPTION_STATIC_SCRATCH_BYTES = 4 << 20


def dr_inception_slim_static(desc, B, H, W, x, w, b, y, stream=None):
    """dr_inception_slim without a workspace argument: the scratch tensor lives in a fixed array
    inside the library (see include/dr.h for the size limit and the sharing rules)."""
    wa = (_P * 3)(*[_ptr(t) for t in w])
    ba = (_P * 3)(*[_ptr(t) for t in b])
    _check(_lib.dr_inception_slim_static(C.byref(desc), B, H, W, _ptr(x), wa, ba, _ptr(y), _stream(stream)),
           "dr_inception_slim_static")


def dr_relu(n, x, y, stream=None):
    _check(_lib.dr_relu(n, _ptr(x), _ptr(y), _stream(stream)), "dr_relu")


def dr_maxpool(B, H, W, Cc, k, s, p, x, y, argmax=None, stream=None):
    _check(_lib.dr_maxpool(B, H, W, Cc, k, s, p, _ptr(x), _ptr(y), _ptr(argmax), _stream(stream)), "dr_maxpool")


def dr_lrn(B, H, W, Cc, size, alpha, beta, k, x, y, stream=None):
    _check(_lib.dr_lrn(B, H, W, Cc, size, alpha, beta, k, _ptr(x), _ptr(y), _stream(stream)), "dr_lrn")


def dr_bn(B, H, W, Cc, x, mean, var, m, eps, gamma, beta, y, stream=None):
    _check(_lib.dr_bn(B, H, W, Cc, _ptr(x), _ptr(mean), _ptr(var), m, eps, _ptr(gamma), _ptr(beta), _ptr(y), _stream(stream)), "dr_bn")


def dr_scale(B, H, W, Cc, x, gamma, beta, y, stream=None):
    _check(_lib.dr_scale(B, H, W, Cc, _ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), _stream(stream)), "dr_scale")


def dr_add(n, a, b, y, stream=None):
    _check(_lib.dr_add(n, _ptr(a), _ptr(b), _ptr(y), _stream(stream)), "dr_add")


def dr_concat(npix, Cc, x, ldc, coff, y, stream=None):
    _check(_lib.dr_concat(npix, Cc, _ptr(x), ldc, coff, _ptr(y), _stream(stream)), "dr_concat")


def dr_avgpool_global(B, H, W, Cc, x, y, stream=None):
    _check(_lib.dr_avgpool_global(B, H, W, Cc, _ptr(x), _ptr(y), _stream(stream)), "dr_avgpool_global")


def dr_set_conv_path(path: int):
    _check(_lib.dr_set_conv_path(path), "dr_set_conv_path")


def dr_last_conv_path() -> int:
    return _lib.dr_last_conv_path()


def dr_device_status():
    """Synchronises; returns (status, info[4])."""
    info = (_I * 4)()
    st = _lib.dr_device_status(info)
    return st, list(info)


def dr_selftest_wait_timeout(limit_cycles: int, stream=None):
    _check(_lib.dr_selftest_wait_timeout(limit_cycles, _stream(stream)), "dr_selftest_wait_timeout")


def dr_launch_count() -> int:
    return int(_lib.dr_launch_count())


def dr_tensor_map_encodes() -> int:
    return int(_lib.dr_tensor_map_encodes())


def dr_conv_plan(desc, B, H, W, workspace_bytes: int = 0) -> dict:
    """How the library would run the layer: kernel path, accumulator-block width and count, CTA pairs, wide tiles."""
    plan = (_I * 8)()
    _check(_lib.dr_conv_plan(C.byref(desc), B, H, W, workspace_bytes, plan), "dr_conv_plan")
    return {"path": PATH_NAMES[plan[0]], "Nt": plan[1], "n_blocks": plan[2], "pair": plan[3], "wide": plan[4]}


class Net:
    """Owner of a ``dr_net*``: same calls as the C API, handle kept for you."""

    _h = None

    def __init__(self, arch: int, mode: int, B: int, H: int = 224, W: int = 224):
        h = _P()
        _check(_lib.dr_net_create(C.byref(h), arch, mode, B, H, W), "dr_net_create")
        self._h = h
        self.arch, self.mode, self.B, self.H, self.W = arch, mode, B, H, W

    def close(self):
        if self._h:
            _lib.dr_net_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def dr_net_num_params(self) -> int:
        return _lib.dr_net_num_params(self._h)

    def dr_net_param_spec(self, idx: int):
        s = dr_param_spec()
        _check(_lib.dr_net_param_spec(self._h, idx, C.byref(s)), "dr_net_param_spec")
        return s.name.decode(), tuple(s.dims), bool(s.is_f32), int(s.count)

    def dr_net_set_param(self, idx: int, dev):
        _check(_lib.dr_net_set_param(self._h, idx, _ptr(dev)), "dr_net_set_param")

    def dr_net_workspace_bytes(self) -> int:
        n = _Z(0)
        _check(_lib.dr_net_workspace_bytes(self._h, C.byref(n)), "dr_net_workspace_bytes")
        return n.value

    def dr_net_activation_bytes(self) -> int:
        n = _Z(0)
        _check(_lib.dr_net_activation_bytes(self._h, C.byref(n)), "dr_net_activation_bytes")
        return n.value

    def dr_net_prepare(self, workspace, stream=None):
        _check(_lib.dr_net_prepare(self._h, _ptr(workspace), _stream(stream)), "dr_net_prepare")

    def dr_net_forward(self, x, workspace, logits, stream=None):
        _check(_lib.dr_net_forward(self._h, _ptr(x), _ptr(workspace), _ptr(logits), _stream(stream)), "dr_net_forward")

    def dr_net_num_layers(self) -> int:
        return _lib.dr_net_num_layers(self._h)

    def dr_net_layer_info(self, layer: int) -> dict:
        li = dr_layer_info()
        _check(_lib.dr_net_layer_info(self._h, layer, C.byref(li)), "dr_net_layer_info")
        return dict(name=li.name.decode(), kind=li.kind, dims=tuple(li.dims), ldc=li.ldc, coff=li.coff,
                    is_f32=bool(li.is_f32), ptr=li.ptr, flops=li.flops, bytes=li.bytes, conv_path=li.conv_path)

    def dr_net_set_timing(self, enabled: bool):
        _check(_lib.dr_net_set_timing(self._h, int(enabled)), "dr_net_set_timing")

    def dr_net_layer_time_us(self, layer: int) -> float:
        us = _F(0)
        _check(_lib.dr_net_layer_time_us(self._h, layer, C.byref(us)), "dr_net_layer_time_us")
        return us.value
