"""ctypes binding of ``include/xenos.h``: same names, argument marshalling only.

Every step of the path (pre-fusion, linking, split, kernels) runs inside ``libxenos.so``;
PyTorch is used by callers for device memory and streams.  There is no CPU fallback: loading
fails loudly when the library cannot be built or found.
"""
from __future__ import annotations

import ctypes
import json
import os
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

XENOS_OK = 0
E_INVALID, E_SHAPE, E_UNSUPPORTED, E_NOT_LINKABLE, E_BAD_SPLIT = -1, -2, -3, -4, -5
E_STATE, E_WORKSPACE, E_CUDA, E_TIMEOUT, E_BOUNDS = -6, -7, -8, -9, -10
OP_CONV, OP_FC, OP_POOL_MAX, OP_POOL_AVG, OP_POOL_GLOBAL_AVG = 1, 2, 3, 4, 5
OP_ADD, OP_CONCAT, OP_RELU, OP_RELU6, OP_BATCHNORM = 6, 7, 8, 9, 10
OP_MUL, OP_MAC, OP_TRANSPOSE, OP_SPLIT, OP_MATMUL = 11, 12, 13, 14, 15
ACT_NONE, ACT_RELU, ACT_RELU6 = 0, 1, 2
DTYPE_F32, DTYPE_BF16 = 0, 1
LAYOUT_NCHW, LAYOUT_NHWC = 0, 1
PRECISION_FP32_CUDA_CORE, PRECISION_BF16_TENSOR = 0, 1

_f32p = ctypes.POINTER(ctypes.c_float)


class HwInfo(ctypes.Structure):
    _fields_ = [("sm_count", ctypes.c_int32), ("smem_bytes_per_cta", ctypes.c_int32),
                ("tmem_columns", ctypes.c_int32), ("l2_bytes", ctypes.c_int64)]


class OpDesc(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("cout", ctypes.c_int32), ("kh", ctypes.c_int32), ("kw", ctypes.c_int32),
                ("stride", ctypes.c_int32), ("pad", ctypes.c_int32), ("groups", ctypes.c_int32), ("act", ctypes.c_int32),
                ("weight", _f32p), ("bias", _f32p), ("bn_gamma", _f32p), ("bn_beta", _f32p), ("bn_mean", _f32p),
                ("bn_var", _f32p), ("bn_eps", ctypes.c_float)]


EXPORTS = ["xenos_graph_create", "xenos_graph_add_input", "xenos_graph_add_op", "xenos_graph_mark_output",
           "xenos_graph_link", "xenos_graph_split", "xenos_graph_search_split", "xenos_graph_compile", "xenos_graph_bind", "xenos_graph_run",
           "xenos_graph_profile", "xenos_graph_run_builtin_scratch", "xenos_graph_status", "xenos_graph_selftest_wait_expiry", "xenos_graph_get_plan", "xenos_graph_launch_count", "xenos_graph_save", "xenos_graph_load", "xenos_graph_destroy",
           "xenos_last_error"]

_lib = None


def lib() -> ctypes.CDLL:
    """Loads (building if stale) the CUDA library; raises if that is impossible."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = ctypes.CDLL(path)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        L.xenos_graph_create.argtypes = [ctypes.POINTER(HwInfo), ctypes.POINTER(vp)]
        L.xenos_graph_add_input.argtypes = [vp, i32, i32, i32, i32, i32, ctypes.POINTER(i32)]
        L.xenos_graph_add_op.argtypes = [vp, ctypes.POINTER(OpDesc), ctypes.POINTER(i32), i32, ctypes.POINTER(i32)]
        L.xenos_graph_mark_output.argtypes = [vp, i32, i32, i32]
        L.xenos_graph_link.argtypes = [vp, ctypes.POINTER(i32), i32]
        L.xenos_graph_split.argtypes = [vp, i32, i32, i32, i32, i32]
        L.xenos_graph_search_split.argtypes = [vp, i32, i32, vp, sz, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, i32, i32,
                                               ctypes.c_char_p, sz, ctypes.POINTER(sz)]
        L.xenos_graph_compile.argtypes = [vp, i32, i32, ctypes.POINTER(sz)]
        L.xenos_graph_bind.argtypes = [vp, vp, sz, vp]
        L.xenos_graph_run.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), vp]
        L.xenos_graph_profile.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, _f32p, i32]
        L.xenos_graph_run_builtin_scratch.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), vp]
        L.xenos_graph_status.argtypes = [vp, vp]
        L.xenos_graph_selftest_wait_expiry.argtypes = [vp, vp]
        L.xenos_graph_get_plan.argtypes = [vp, ctypes.c_char_p, sz, ctypes.POINTER(sz)]
        L.xenos_graph_launch_count.argtypes = [vp, ctypes.POINTER(i32)]
        L.xenos_graph_save.argtypes = [vp, vp, sz, ctypes.POINTER(sz)]
        L.xenos_graph_load.argtypes = [vp, sz, ctypes.POINTER(vp), ctypes.POINTER(sz)]
        L.xenos_graph_destroy.argtypes = [vp]
        L.xenos_last_error.argtypes = [vp]
        L.xenos_last_error.restype = ctypes.c_char_p
        for n in EXPORTS[:-1]:
            getattr(L, n).restype = i32
        _lib = L
    return _lib


class XenosError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"xenos error {code}: {msg}")
        self.code = code


def _fp(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_f32p)


class Graph:
    """One ``xenos_graph_t``; methods mirror the C entry points one to one."""

    def __init__(self, hw: Optional[HwInfo] = None):
        self._h = ctypes.c_void_p()
        rc = lib().xenos_graph_create(ctypes.byref(hw) if hw is not None else None, ctypes.byref(self._h))
        if rc != XENOS_OK:
            raise XenosError(rc, lib().xenos_last_error(None).decode())
        self._keep: List[np.ndarray] = []

    def _check(self, rc: int):
        if rc != XENOS_OK:
            raise XenosError(rc, lib().xenos_last_error(self._h).decode())

    def add_input(self, dtype: int, layout: int, c: int, h: int, w: int) -> int:
        t = ctypes.c_int32()
        self._check(lib().xenos_graph_add_input(self._h, dtype, layout, c, h, w, ctypes.byref(t)))
        return t.value

    def add_op(self, kind: int, inputs: Sequence[int], cout=0, k=0, stride=1, pad=0, groups=1, act=ACT_NONE,
               weight=None, bias=None, bn=None, bn_eps=1e-5) -> int:
        d = OpDesc()
        d.kind, d.cout, d.kh, d.kw, d.stride, d.pad, d.groups, d.act = kind, cout, k, k, stride, pad, groups, act
        arrs = []
        def c32(a):
            if a is None:
                return None
            a = np.ascontiguousarray(a, dtype=np.float32)
            arrs.append(a)
            return a
        d.weight, d.bias = _fp(c32(weight)), _fp(c32(bias))
        if bn is not None:
            d.bn_gamma, d.bn_beta, d.bn_mean, d.bn_var = (_fp(c32(x)) for x in bn)
        d.bn_eps = bn_eps
        ins = (ctypes.c_int32 * len(inputs))(*inputs)
        t = ctypes.c_int32()
        self._check(lib().xenos_graph_add_op(self._h, ctypes.byref(d), ins, len(inputs), ctypes.byref(t)))
        return t.value

    def mark_output(self, tensor: int, dtype: int, layout: int):
        self._check(lib().xenos_graph_mark_output(self._h, tensor, dtype, layout))

    def link(self, ops: Sequence[int] = ()):
        arr = (ctypes.c_int32 * max(1, len(ops)))(*ops)
        self._check(lib().xenos_graph_link(self._h, arr, len(ops)))

    def split(self, op: int = -1, parts_outc=0, parts_h=0, parts_w=0, parts_k=1):
        self._check(lib().xenos_graph_split(self._h, op, parts_outc, parts_h, parts_w, parts_k))

    def search_split(self, max_batch: int, precision: int, workspace_ptr: int, nbytes: int, inputs: Sequence[int],
                     outputs: Sequence[int], stream: int = 0, max_trials: int = 8, repeats: int = 5) -> dict:
        ins = (ctypes.c_void_p * len(inputs))(*inputs)
        outs = (ctypes.c_void_p * len(outputs))(*outputs)
        need = ctypes.c_size_t()
        cap = 1 << 20
        buf = ctypes.create_string_buffer(cap)
        self._check(lib().xenos_graph_search_split(self._h, max_batch, precision, workspace_ptr, nbytes, ins, outs, stream,
                                                   max_trials, repeats, buf, cap, ctypes.byref(need)))
        return json.loads(buf.value.decode())

    def compile(self, max_batch: int, precision: int) -> int:
        n = ctypes.c_size_t()
        self._check(lib().xenos_graph_compile(self._h, max_batch, precision, ctypes.byref(n)))
        return n.value

    def bind(self, workspace_ptr: int, nbytes: int, stream: int = 0):
        self._check(lib().xenos_graph_bind(self._h, ctypes.c_void_p(workspace_ptr), nbytes, ctypes.c_void_p(stream)))

    def run(self, batch: int, inputs: Sequence[int], outputs: Sequence[int], stream: int = 0):
        ia = (ctypes.c_void_p * len(inputs))(*inputs)
        oa = (ctypes.c_void_p * len(outputs))(*outputs)
        self._check(lib().xenos_graph_run(self._h, batch, ia, oa, ctypes.c_void_p(stream)))

    def profile(self, batch: int, inputs: Sequence[int], outputs: Sequence[int], stream: int = 0) -> List[float]:
        n = self.launch_count()
        ms = (ctypes.c_float * n)()
        ia = (ctypes.c_void_p * len(inputs))(*inputs)
        oa = (ctypes.c_void_p * len(outputs))(*outputs)
        self._check(lib().xenos_graph_profile(self._h, batch, ia, oa, ctypes.c_void_p(stream), ms, n))
        return list(ms)

    def run_builtin_scratch(self, batch: int, inputs: Sequence[int], outputs: Sequence[int], stream: int = 0):
        """Inference with the library's built-in 16 MiB workspace instead of a bound one (synchronous)."""
        ia = (ctypes.c_void_p * len(inputs))(*inputs)
        oa = (ctypes.c_void_p * len(outputs))(*outputs)
        self._check(lib().xenos_graph_run_builtin_scratch(self._h, batch, ia, oa, ctypes.c_void_p(stream)))

    def status(self, stream: int = 0):
        self._check(lib().xenos_graph_status(self._h, ctypes.c_void_p(stream)))

    def selftest_wait_expiry(self, stream: int = 0):
        self._check(lib().xenos_graph_selftest_wait_expiry(self._h, ctypes.c_void_p(stream)))

    def plan(self) -> dict:
        n = ctypes.c_size_t()
        self._check(lib().xenos_graph_get_plan(self._h, None, 0, ctypes.byref(n)))
        buf = ctypes.create_string_buffer(n.value)
        self._check(lib().xenos_graph_get_plan(self._h, buf, n.value, ctypes.byref(n)))
        return json.loads(buf.value.decode())

    def plan_text(self) -> str:
        n = ctypes.c_size_t()
        self._check(lib().xenos_graph_get_plan(self._h, None, 0, ctypes.byref(n)))
        buf = ctypes.create_string_buffer(n.value)
        self._check(lib().xenos_graph_get_plan(self._h, buf, n.value, ctypes.byref(n)))
        return buf.value.decode()

    def save(self) -> bytes:
        n = ctypes.c_size_t()
        self._check(lib().xenos_graph_save(self._h, None, 0, ctypes.byref(n)))
        buf = ctypes.create_string_buffer(n.value)
        self._check(lib().xenos_graph_save(self._h, buf, n.value, ctypes.byref(n)))
        return buf.raw[:n.value]

    @classmethod
    def load(cls, image: bytes):
        """Returns (graph, workspace_bytes); workspace_bytes is 0 when the saved graph had not been compiled."""
        g = cls.__new__(cls)
        g._h = ctypes.c_void_p()
        g._keep = []
        n = ctypes.c_size_t()
        buf = ctypes.create_string_buffer(image, len(image))
        rc = lib().xenos_graph_load(buf, len(image), ctypes.byref(g._h), ctypes.byref(n))
        if rc != XENOS_OK:
            raise XenosError(rc, lib().xenos_last_error(None).decode())
        return g, n.value

    def launch_count(self) -> int:
        n = ctypes.c_int32()
        self._check(lib().xenos_graph_launch_count(self._h, ctypes.byref(n)))
        return n.value

    def destroy(self):
        if self._h:
            lib().xenos_graph_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
