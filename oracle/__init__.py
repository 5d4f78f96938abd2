"""CPU oracle (test infrastructure, never on the product path).

Thin ctypes wrappers over ``xoracle.c``: every operator of the paper's Table 3 that the CNN
workloads use, run one at a time on NCHW fp32 numpy arrays.  Nothing here imports or is
imported by the CUDA library.  ``build()`` compiles the C file with gcc; it is called lazily
on first use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xoracle.c")
_LIB = os.path.join(_HERE, "libxoracle.so")
_lock = threading.Lock()
_lib = None

_f32p = ctypes.POINTER(ctypes.c_float)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the oracle.  -ffp-contract=off keeps every a*b+c as two rounded operations, so
    the same expression gives the same bits wherever it appears."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                   "-fvisibility=hidden", "-o", _LIB, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.xo_num_threads.restype = ctypes.c_int
        L.xo_out_dim.restype = ctypes.c_int
        L.xo_chain_tiled.restype = ctypes.c_int
        L.xo_stage_struct_size.restype = ctypes.c_size_t
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(_f32p)


def _c(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def num_threads() -> int:
    return int(lib().xo_num_threads())


def set_num_threads(n: int) -> None:
    lib().xo_set_num_threads(ctypes.c_int(n))


def out_dim(i: int, k: int, stride: int, pad: int) -> int:
    return int(lib().xo_out_dim(i, k, stride, pad))


def conv2d(x, w, bias=None, stride=1, pad=0, groups=1):
    x, w, bias = _c(x), _c(w), _c(bias)
    N, C, H, W = x.shape
    K, Cg, R, S = w.shape
    assert Cg * groups == C and K % groups == 0
    P, Q = out_dim(H, R, stride, pad), out_dim(W, S, stride, pad)
    y = np.empty((N, K, P, Q), np.float32)
    lib().xo_conv2d(_p(x), N, C, H, W, _p(w), K, R, S, stride, pad, groups, _p(bias), _p(y))
    return y


def batchnorm(x, gamma, beta, mean, var, eps=1e-5):
    x = _c(x)
    N, C = x.shape[:2]
    HW = int(np.prod(x.shape[2:])) if x.ndim > 2 else 1
    y = np.empty_like(x)
    lib().xo_batchnorm(_p(x), N, C, HW, _p(_c(gamma)), _p(_c(beta)), _p(_c(mean)), _p(_c(var)),
                       ctypes.c_float(eps), _p(y))
    return y


def relu(x):
    x = _c(x)
    y = np.empty_like(x)
    lib().xo_relu(_p(x), ctypes.c_size_t(x.size), _p(y))
    return y


def relu6(x):
    x = _c(x)
    y = np.empty_like(x)
    lib().xo_relu6(_p(x), ctypes.c_size_t(x.size), _p(y))
    return y


def maxpool(x, k, stride, pad=0):
    x = _c(x)
    N, C, H, W = x.shape
    y = np.empty((N, C, out_dim(H, k, stride, pad), out_dim(W, k, stride, pad)), np.float32)
    lib().xo_maxpool(_p(x), N, C, H, W, k, stride, pad, _p(y))
    return y


def avgpool(x, k, stride, pad=0):
    x = _c(x)
    N, C, H, W = x.shape
    y = np.empty((N, C, out_dim(H, k, stride, pad), out_dim(W, k, stride, pad)), np.float32)
    lib().xo_avgpool(_p(x), N, C, H, W, k, stride, pad, _p(y))
    return y


def global_avgpool(x):
    x = _c(x)
    N, C, H, W = x.shape
    y = np.empty((N, C), np.float32)
    lib().xo_global_avgpool(_p(x), N, C, H * W, _p(y))
    return y


def add(a, b):
    a, b = _c(a), _c(b)
    assert a.shape == b.shape
    y = np.empty_like(a)
    lib().xo_add(_p(a), _p(b), ctypes.c_size_t(a.size), _p(y))
    return y


def concat(xs):
    xs = [_c(x) for x in xs]
    N, _, H, W = xs[0].shape
    ctot = sum(x.shape[1] for x in xs)
    y = np.empty((N, ctot, H, W), np.float32)
    off = 0
    for x in xs:
        assert x.shape[0] == N and x.shape[2:] == (H, W)
        lib().xo_concat_part(_p(x), N, x.shape[1], H * W, ctot, off, _p(y))
        off += x.shape[1]
    return y


def mul(a, b):
    a, b = _c(a), _c(b)
    assert a.shape == b.shape
    y = np.empty_like(a)
    lib().xo_mul(_p(a), _p(b), ctypes.c_size_t(a.size), _p(y))
    return y


def mac(a, b, c):
    a, b, c = _c(a), _c(b), _c(c)
    assert a.shape == b.shape == c.shape
    y = np.empty_like(a)
    lib().xo_mac(_p(a), _p(b), _p(c), ctypes.c_size_t(a.size), _p(y))
    return y


def transpose(x):
    """Matrix transpose per image: (N, C, H, 1) -> (N, H, C, 1)."""
    x = _c(x)
    N, C, H, W = x.shape
    assert W == 1
    y = np.empty((N, H, C, 1), np.float32)
    lib().xo_transpose(_p(x), N, C, H, _p(y))
    return y


def split_part(x, first, count):
    x = _c(x)
    N, C, H, W = x.shape
    assert 0 <= first and first + count <= C
    y = np.empty((N, count, H, W), np.float32)
    lib().xo_split_part(_p(x), N, count, H * W, C, first, _p(y))
    return y


def matmul(a, b, bias=None):
    """a: (N, K, R, 1) matrix per image (R rows of K columns) or (N, K) vectors; b: (K, M) constant."""
    a, b, bias = _c(a), _c(b), _c(bias)
    vec = a.ndim == 2
    N, K = a.shape[0], a.shape[1]
    R = 1 if vec else a.shape[2]
    assert b.shape[0] == K and (vec or a.shape[3] == 1)
    M = b.shape[1]
    y = np.empty((N, M) if vec else (N, M, R, 1), np.float32)
    lib().xo_matmul(_p(a), N, K, R, _p(b), M, _p(bias), _p(y))
    return y


def fc(x, w, bias=None):
    x, w, bias = _c(x), _c(w), _c(bias)
    N, C = x.shape
    K = w.shape[0]
    assert w.shape[1] == C
    y = np.empty((N, K), np.float32)
    lib().xo_fc(_p(x), N, C, _p(w), K, _p(bias), _p(y))
    return y


def round_bf16(x):
    x = _c(x)
    y = np.empty_like(x)
    lib().xo_round_bf16(_p(x), ctypes.c_size_t(x.size), _p(y))
    return y


class _Stage(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("cout", ctypes.c_int32), ("k", ctypes.c_int32),
                ("stride", ctypes.c_int32), ("pad", ctypes.c_int32), ("groups", ctypes.c_int32),
                ("act", ctypes.c_int32), ("has_bn", ctypes.c_int32),
                ("w", _f32p), ("bias", _f32p), ("gamma", _f32p), ("beta", _f32p),
                ("mean", _f32p), ("var", _f32p), ("eps", ctypes.c_float)]


_ACT = {None: 0, "none": 0, "relu": 1, "relu6": 2}


def chain_tiled(x, stages, th, tw, want_halo=False):
    """Linked evaluation of a chain, one output tile (th x tw of the last stage) at a time.

    ``stages``: list of dicts; conv: {kind:'conv', w, bias?, stride, pad, groups, bn?:(g,b,m,v,eps),
    act?}; pool: {kind:'maxpool'|'avgpool', k, stride, pad}.
    """
    assert ctypes.sizeof(_Stage) == lib().xo_stage_struct_size()
    x = _c(x)
    N, C, H, W = x.shape
    arr = (_Stage * len(stages))()
    keep = []
    c, h, w_ = C, H, W
    for i, s in enumerate(stages):
        st = arr[i]
        if s["kind"] == "conv":
            wt = _c(s["w"]); keep.append(wt)
            st.kind, st.cout, st.k = 0, wt.shape[0], wt.shape[2]
            st.stride, st.pad, st.groups = s.get("stride", 1), s.get("pad", 0), s.get("groups", 1)
            st.act = _ACT[s.get("act")]
            st.w = _p(wt)
            b = _c(s.get("bias")); keep.append(b); st.bias = _p(b)
            bn = s.get("bn")
            st.has_bn = 1 if bn else 0
            if bn:
                g, be, m, v = (_c(t) for t in bn[:4]); keep += [g, be, m, v]
                st.gamma, st.beta, st.mean, st.var = _p(g), _p(be), _p(m), _p(v)
                st.eps = bn[4] if len(bn) > 4 else 1e-5
            c = wt.shape[0]
        else:
            st.kind = 1 if s["kind"] == "maxpool" else 2
            st.k, st.stride, st.pad, st.groups = s["k"], s["stride"], s.get("pad", 0), 1
        h, w_ = out_dim(h, st.k, st.stride, st.pad), out_dim(w_, st.k, st.stride, st.pad)
    y = np.empty((N, c, h, w_), np.float32)
    halo = np.zeros((len(stages), 4), np.int32) if want_halo else None
    rc = lib().xo_chain_tiled(_p(x), N, C, H, W, arr, len(stages), th, tw, _p(y),
                              None if halo is None else halo.ctypes.data_as(_i32p))
    if rc != 0:
        raise RuntimeError("xo_chain_tiled failed")
    return (y, halo) if want_halo else y
