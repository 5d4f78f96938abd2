"""Graph interpreter over the CPU oracle (test infrastructure, never on the product path).

Walks the operator records of a workload graph in order and evaluates each with the plain
NCHW fp32 definition from ``xoracle.c``: one operator at a time, BatchNorm un-folded, every
intermediate a full tensor.  That is the "original model" the paper's optimised model must be
equivalent to (Section 3).
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

import oracle as xo


def run_graph(spec, params, x: np.ndarray, keep: bool = False, bf16_emulate: bool = False):
    """Evaluate ``spec`` on input ``x`` (NCHW fp32).  Returns the output array, or the dict of
    all tensors when ``keep``.  ``bf16_emulate`` (diagnostic) rounds the input and every op
    output to bf16 so that precision drift can be told apart from an indexing error."""
    rnd = xo.round_bf16 if bf16_emulate else (lambda a: a)
    t: Dict[str, np.ndarray] = {"input": rnd(np.ascontiguousarray(x, np.float32))}
    for o in spec.ops:
        ins = [t[n] for n in o["inputs"]]
        p = params.get(o["name"], {})
        k = o["kind"]
        if k == "conv":
            y = xo.conv2d(ins[0], p["w"], p.get("b"), o["stride"], o["pad"], o["groups"])
        elif k == "bn":
            y = xo.batchnorm(ins[0], p["gamma"], p["beta"], p["mean"], p["var"], 1e-5)
        elif k == "relu":
            y = xo.relu(ins[0])
        elif k == "relu6":
            y = xo.relu6(ins[0])
        elif k == "maxpool":
            y = xo.maxpool(ins[0], o["k"], o["stride"], o["pad"])
        elif k == "avgpool":
            y = xo.avgpool(ins[0], o["k"], o["stride"], o["pad"])
        elif k == "gap":
            y = xo.global_avgpool(ins[0])
        elif k == "add":
            y = xo.add(ins[0], ins[1])
        elif k == "concat":
            y = xo.concat(ins)
        elif k == "fc":
            y = xo.fc(ins[0], p["w"], p.get("b"))
        elif k == "mul":
            y = xo.mul(ins[0], ins[1])
        elif k == "mac":
            y = xo.mac(ins[0], ins[1], ins[2])
        elif k == "transpose":
            y = xo.transpose(ins[0])
        elif k == "split":
            y = xo.split_part(ins[0], o["first"], o["cout"])
        elif k == "matmul":
            y = xo.matmul(ins[0], p["w"], p.get("b"))
        else:
            raise ValueError(k)
        # BatchNorm and activation follow their conv inside one fused operator on the device,
        # so only the end of such a group is a stored (rounded) tensor in the emulation.
        t[o["out"]] = y
        if bf16_emulate and not _feeds_fused_tail(spec, o):
            t[o["out"]] = rnd(y)
    return t if keep else t[spec.output]


def _feeds_fused_tail(spec, o) -> bool:
    """True when the only consumer of ``o`` is a bn/relu/relu6 record (or add->relu tail)."""
    cons = [c for c in spec.ops if o["out"] in c["inputs"]]
    if len(cons) != 1:
        return False
    ck = cons[0]["kind"]
    if o["kind"] in ("conv", "bn") and ck in ("bn", "relu", "relu6"):
        return True
    if o["kind"] in ("conv", "bn") and ck == "add":
        return True
    if o["kind"] == "add" and ck in ("relu", "relu6"):
        return True
    return False
