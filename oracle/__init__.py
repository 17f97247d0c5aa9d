"""CPU checker (test infrastructure only): ctypes front end of ``dr_oracle.cpp``.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  The CUDA library never does, and this package never imports the CUDA
library or its Python binding.

All tensors are NHWC ``float64`` numpy arrays; filters are ``[Cout][k][k][Cin]``.
Each function states the passage of the paper it follows in ``dr_oracle.cpp``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dr_oracle.cpp")
_LIB = os.path.join(_HERE, "libdr_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with g++ (OpenMP over output pixels only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c++17",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_out_size.restype = ctypes.c_int
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _dn(a):
    if a is None:
        return None, None
    return _d(a)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def out_size(n: int, k: int, stride: int, pad: int) -> int:
    return int(lib().orc_out_size(int(n), int(k), int(stride), int(pad)))


def conv2d(x, w, bias=None, stride=1, pad=0):
    B, H, W, Cin = x.shape
    Cout, k, k2, Cin2 = w.shape
    assert k == k2 and Cin == Cin2
    x, px = _d(x); w, pw = _d(w); bias, pb = _dn(bias)
    Ho, Wo = out_size(H, k, stride, pad), out_size(W, k, stride, pad)
    y = np.empty((B, Ho, Wo, Cout), np.float64)
    lib().orc_conv2d(B, H, W, Cin, px, k, stride, pad, Cout, pw, pb, _d(y)[1])
    return y


def conv2d_grouped(x, w, bias=None, stride=1, pad=0, groups=1):
    """Grouped convolution by its definition: group g convolves input channels [g*Cin_g, (g+1)*Cin_g) with filters
    [g*Cout_g, (g+1)*Cout_g) and the group outputs are concatenated along channels.  w: [Cout][k][k][Cin_g]."""
    Cout, Cin_g = w.shape[0], w.shape[3]
    assert x.shape[3] == Cin_g * groups and Cout % groups == 0
    cg = Cout // groups
    parts = [conv2d(np.ascontiguousarray(x[..., g * Cin_g:(g + 1) * Cin_g]), np.ascontiguousarray(w[g * cg:(g + 1) * cg]),
                    None if bias is None else np.ascontiguousarray(np.asarray(bias)[g * cg:(g + 1) * cg]), stride, pad)
             for g in range(groups)]
    return concat(parts)


def batchnorm(x, mu, sigma2, m=1.0, eps=0.0):
    C = x.shape[-1]
    x, px = _d(x); mu, pm = _d(mu); sigma2, pv = _d(sigma2)
    y = np.empty_like(x)
    lib().orc_batchnorm(ctypes.c_long(x.size // C), C, px, pm, pv, ctypes.c_double(m),
                        ctypes.c_double(eps), _d(y)[1])
    return y


def scale(x, gamma, beta):
    C = x.shape[-1]
    x, px = _d(x); gamma, pg = _d(gamma); beta, pb = _d(beta)
    y = np.empty_like(x)
    lib().orc_scale(ctypes.c_long(x.size // C), C, px, pg, pb, _d(y)[1])
    return y


def relu(x):
    x, px = _d(x)
    y = np.empty_like(x)
    lib().orc_relu(ctypes.c_long(x.size), px, _d(y)[1])
    return y


def maxpool(x, k=3, stride=2, pad=1):
    """Returns (y, argmax); argmax is int32, flat h*W+w in the input plane."""
    B, H, W, C = x.shape
    x, px = _d(x)
    Ho, Wo = out_size(H, k, stride, pad), out_size(W, k, stride, pad)
    y = np.empty((B, Ho, Wo, C), np.float64)
    am = np.empty((B, Ho, Wo, C), np.int32)
    lib().orc_maxpool(B, H, W, C, k, stride, pad, px, _d(y)[1],
                      am.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    return y, am


def lrn(x, size=5, alpha=1e-4, beta=0.75, k=1.0):
    C = x.shape[-1]
    x, px = _d(x)
    y = np.empty_like(x)
    lib().orc_lrn(ctypes.c_long(x.size // C), C, size, ctypes.c_double(alpha), ctypes.c_double(beta),
                  ctypes.c_double(k), px, _d(y)[1])
    return y


def add(a, b):
    a, pa = _d(a); b, pb = _d(b)
    assert a.shape == b.shape
    y = np.empty_like(a)
    lib().orc_add(ctypes.c_long(a.size), pa, pb, _d(y)[1])
    return y


def concat(parts):
    """Channel concatenation of NHWC tensors, one branch at a time."""
    ldc = sum(p.shape[-1] for p in parts)
    y = np.empty(parts[0].shape[:-1] + (ldc,), np.float64)
    off = 0
    for p in parts:
        p, pp = _d(p)
        C = p.shape[-1]
        lib().orc_concat_into(ctypes.c_long(p.size // C), C, pp, ldc, off, _d(y)[1])
        off += C
    return y


def avgpool_global(x):
    B, H, W, C = x.shape
    x, px = _d(x)
    y = np.empty((B, 1, 1, C), np.float64)
    lib().orc_avgpool_global(B, H, W, C, px, _d(y)[1])
    return y


def fold_bn(w, b, mu, sigma2, m, eps, gamma, beta):
    """Lemma 2 closed form; returns (W~, B~) in float64."""
    Cout = w.shape[0]
    K = w.size // Cout
    w, pw = _d(w); b, pb = _dn(b); mu, pm = _d(mu); sigma2, pv = _d(sigma2)
    gamma, pg = _d(gamma); beta, pbe = _d(beta)
    wo = np.empty_like(w); bo = np.empty(Cout, np.float64)
    lib().orc_fold_bn(Cout, ctypes.c_long(K), pw, pb, pm, pv, ctypes.c_double(m), ctypes.c_double(eps),
                      pg, pbe, _d(wo)[1], _d(bo)[1])
    return wo, bo


def embed_filter(w_small, kb, w_big=None, joff=0):
    """Zero-embed [Cout][ks][ks][Cin] at the centre of kb x kb filters [joff, joff+Cout) of w_big."""
    Cout, ks, _, Cin = w_small.shape
    w_small, ps = _d(w_small)
    if w_big is None:
        w_big = np.zeros((Cout, kb, kb, Cin), np.float64)
    assert w_big.dtype == np.float64 and w_big.flags.c_contiguous
    lib().orc_embed_filter(Cout, Cin, ks, kb, ps, joff, _d(w_big)[1])
    return w_big


def round_bf16(x):
    x, px = _d(x)
    y = np.empty_like(x)
    lib().orc_round_bf16(ctypes.c_long(x.size), px, _d(y)[1])
    return y
