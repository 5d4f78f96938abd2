"""Feeds a workload graph (plain operator records) to the library's C API through its Python binding.

Harness code: it knows the record format of ``xenos_workloads.graphs`` and calls one ``add_op`` per
record; it holds no operator arithmetic.  Used by the tests and by ``bench.py``.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np


def graph_from_spec(spec, params: Dict[str, Dict[str, np.ndarray]], in_dtype=None, in_layout=None, hw=None):
    """Returns (Graph, {tensor name: id}) for the records of ``spec``."""
    from paper_2302_00282_b200 import binding as xb
    kind = {"mul": xb.OP_MUL, "mac": xb.OP_MAC, "transpose": xb.OP_TRANSPOSE, "maxpool": xb.OP_POOL_MAX, "avgpool": xb.OP_POOL_AVG, "gap": xb.OP_POOL_GLOBAL_AVG, "add": xb.OP_ADD,
            "concat": xb.OP_CONCAT, "relu": xb.OP_RELU, "relu6": xb.OP_RELU6}
    in_dtype = xb.DTYPE_F32 if in_dtype is None else in_dtype
    in_layout = xb.LAYOUT_NCHW if in_layout is None else in_layout
    g = xb.Graph(hw)
    ids = {"input": g.add_input(in_dtype, in_layout, *spec.in_shape)}
    for o in spec.ops:
        ins = [ids[n] for n in o["inputs"]]
        p = params.get(o["name"], {})
        k = o["kind"]
        if k == "conv":
            t = g.add_op(xb.OP_CONV, ins, cout=o["cout"], k=o["k"], stride=o["stride"], pad=o["pad"], groups=o["groups"],
                         weight=p["w"], bias=p.get("b"))
        elif k == "fc":
            t = g.add_op(xb.OP_FC, ins, cout=o["cout"], k=1, weight=p["w"], bias=p.get("b"))
        elif k == "matmul":
            t = g.add_op(xb.OP_MATMUL, ins, cout=o["cout"], k=1, weight=p["w"], bias=p.get("b"))
        elif k == "split":
            t = g.add_op(xb.OP_SPLIT, ins, cout=o["cout"], pad=o["first"])
        elif k == "bn":
            t = g.add_op(xb.OP_BATCHNORM, ins, bn=(p["gamma"], p["beta"], p["mean"], p["var"]), bn_eps=1e-5)
        elif k in ("maxpool", "avgpool"):
            t = g.add_op(kind[k], ins, k=o["k"], stride=o["stride"], pad=o["pad"])
        else:
            t = g.add_op(kind[k], ins)
        ids[o["out"]] = t
    fp32 = spec.precision == "fp32"
    vec = len(spec.shapes[spec.output]) == 1
    g.mark_output(ids[spec.output], xb.DTYPE_F32 if (fp32 or vec) else xb.DTYPE_BF16,
                  xb.LAYOUT_NCHW if (fp32 or vec) else xb.LAYOUT_NHWC)
    return g, ids
