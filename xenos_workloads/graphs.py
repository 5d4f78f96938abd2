"""Synthetic CNN graphs shaped like the paper's benchmark models, as plain data.

A graph is a list of operator records (dicts) over named tensors; it holds shapes and
hyper-parameters only, no arithmetic.  The CPU oracle's interpreter and the CUDA library's
Python binding both consume these records, and ``make_params`` draws the weights from the
seeded generator, so both sides see identical inputs.

The paper evaluates MobileNet, SqueezeNet and ResNet18 among its seven models (Section 7.1)
without printing their definitions; the graphs here take those models' published shapes and
stand in for them.  Convs followed by BatchNorm carry no conv bias; BatchNorm and activation
are separate records so that the Conv-Bn-Relu pre-fusion (Section 4.3) has work to do.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

from . import gen


def out_dim(i: int, k: int, stride: int, pad: int) -> int:
    return (i + 2 * pad - k) // stride + 1


@dataclass
class GraphSpec:
    name: str
    in_shape: Tuple[int, int, int]                 # (C, H, W) of the single input "input"
    ops: List[dict] = field(default_factory=list)
    shapes: Dict[str, Tuple[int, ...]] = field(default_factory=dict)   # per tensor: (C,H,W) or (C,)
    output: str = ""
    precision: str = "bf16"                        # "fp32" or "bf16"

    def __post_init__(self):
        self.shapes["input"] = tuple(self.in_shape)

    # ---- builders; each appends one record and returns the output tensor name -------------
    def _add(self, rec: dict, shape) -> str:
        rec["out"] = rec["name"]
        self.ops.append(rec)
        self.shapes[rec["name"]] = tuple(shape)
        self.output = rec["name"]
        return rec["name"]

    def conv(self, name, x, cout, k, stride=1, pad=0, groups=1, bias=False) -> str:
        c, h, w = self.shapes[x]
        return self._add(dict(name=name, kind="conv", inputs=[x], cin=c, cout=cout, k=k, stride=stride,
                              pad=pad, groups=groups, bias=bias),
                         (cout, out_dim(h, k, stride, pad), out_dim(w, k, stride, pad)))

    def bn(self, name, x) -> str:
        return self._add(dict(name=name, kind="bn", inputs=[x], c=self.shapes[x][0]), self.shapes[x])

    def act(self, name, x, kind) -> str:
        return self._add(dict(name=name, kind=kind, inputs=[x]), self.shapes[x])

    def pool(self, name, x, kind, k, stride, pad=0) -> str:
        c, h, w = self.shapes[x]
        return self._add(dict(name=name, kind=kind, inputs=[x], k=k, stride=stride, pad=pad),
                         (c, out_dim(h, k, stride, pad), out_dim(w, k, stride, pad)))

    def gap(self, name, x) -> str:
        return self._add(dict(name=name, kind="gap", inputs=[x]), (self.shapes[x][0],))

    def add(self, name, a, b) -> str:
        assert self.shapes[a] == self.shapes[b]
        return self._add(dict(name=name, kind="add", inputs=[a, b]), self.shapes[a])

    def concat(self, name, xs) -> str:
        c = sum(self.shapes[x][0] for x in xs)
        return self._add(dict(name=name, kind="concat", inputs=list(xs)), (c,) + self.shapes[xs[0]][1:])

    def mul(self, name, a, b) -> str:
        assert self.shapes[a] == self.shapes[b]
        return self._add(dict(name=name, kind="mul", inputs=[a, b]), self.shapes[a])

    def mac(self, name, a, b, c) -> str:
        assert self.shapes[a] == self.shapes[b] == self.shapes[c]
        return self._add(dict(name=name, kind="mac", inputs=[a, b, c]), self.shapes[a])

    def transpose(self, name, x) -> str:
        c, h, w = self.shapes[x]
        assert w == 1
        return self._add(dict(name=name, kind="transpose", inputs=[x]), (h, c, 1))

    def split(self, name, x, first, cout) -> str:
        c, h, w = self.shapes[x]
        assert first + cout <= c
        return self._add(dict(name=name, kind="split", inputs=[x], first=first, cout=cout), (cout, h, w))

    def matmul(self, name, x, cout, bias=False) -> str:
        """x (K columns) times a constant [K][cout] matrix."""
        sh = self.shapes[x]
        return self._add(dict(name=name, kind="matmul", inputs=[x], cin=sh[0], cout=cout, bias=bias),
                         (cout,) + tuple(sh[1:]))

    def fc(self, name, x, cout, bias=True) -> str:
        return self._add(dict(name=name, kind="fc", inputs=[x], cin=self.shapes[x][0], cout=cout, bias=bias),
                         (cout,))

    # ---- composite helpers ------------------------------------------------------------------
    def cbr(self, name, x, cout, k, stride=1, pad=0, groups=1, act="relu", bn=True, bias=False) -> str:
        y = self.conv(name, x, cout, k, stride, pad, groups, bias=bias)
        if bn:
            y = self.bn(name + ".bn", y)
        if act:
            y = self.act(name + "." + act, y, act)
        return y

    def macs(self) -> int:
        """Multiply-accumulates per image."""
        t = 0
        for o in self.ops:
            if o["kind"] == "conv":
                _, p, q = self.shapes[o["out"]]
                t += p * q * o["cout"] * (o["cin"] // o["groups"]) * o["k"] * o["k"]
            elif o["kind"] == "fc":
                t += o["cin"] * o["cout"]
        return t


def make_params(spec: GraphSpec, seed: int = gen.DEFAULT_SEED) -> Dict[str, Dict[str, np.ndarray]]:
    """Weights for every parametrised record, tensor ids in graph-construction order.

    conv / fc weights ~ N(0, 2 / fan_in), fan_in = (Cin / groups) * k * k (fc: Cin);
    biases ~ U[-0.1, 0.1]; BatchNorm gamma ~ U[0.5, 1.5], beta ~ U[-0.1, 0.1],
    running mean ~ N(0, 0.1) (0.1 is the standard deviation), running var ~ U[0.5, 1.5].
    Tensor id 0 is reserved for the input image.
    """
    tid = 1
    out: Dict[str, Dict[str, np.ndarray]] = {}
    for o in spec.ops:
        p: Dict[str, np.ndarray] = {}
        if o["kind"] == "conv":
            cg = o["cin"] // o["groups"]
            fan_in = cg * o["k"] * o["k"]
            p["w"] = gen.normal(seed, tid, (o["cout"], cg, o["k"], o["k"]), 0.0, float(np.sqrt(2.0 / fan_in)))
            tid += 1
            if o["bias"]:
                p["b"] = gen.uniform(seed, tid, (o["cout"],), -0.1, 0.1)
            tid += 1
        elif o["kind"] == "matmul":
            p["w"] = gen.normal(seed, tid, (o["cin"], o["cout"]), 0.0, float(np.sqrt(2.0 / o["cin"])))
            tid += 1
            if o["bias"]:
                p["b"] = gen.uniform(seed, tid, (o["cout"],), -0.1, 0.1)
            tid += 1
        elif o["kind"] == "fc":
            p["w"] = gen.normal(seed, tid, (o["cout"], o["cin"]), 0.0, float(np.sqrt(2.0 / o["cin"])))
            tid += 1
            if o["bias"]:
                p["b"] = gen.uniform(seed, tid, (o["cout"],), -0.1, 0.1)
            tid += 1
        elif o["kind"] == "bn":
            c = o["c"]
            p["gamma"] = gen.uniform(seed, tid, (c,), 0.5, 1.5)
            p["beta"] = gen.uniform(seed, tid + 1, (c,), -0.1, 0.1)
            p["mean"] = gen.normal(seed, tid + 2, (c,), 0.0, 0.1)
            p["var"] = gen.uniform(seed, tid + 3, (c,), 0.5, 1.5)
            tid += 4
        if p:
            out[o["name"]] = p
    return out


def make_input(spec: GraphSpec, batch: int, seed: int = gen.DEFAULT_SEED) -> np.ndarray:
    """Input images ~ U[-1, 1], NCHW fp32."""
    return gen.uniform(seed, 0, (batch,) + tuple(spec.in_shape), -1.0, 1.0)


# ------------------------------------------------------------------------------------------------
# The five workload graphs
# ------------------------------------------------------------------------------------------------
def single_chain(hw: int = 32, cin: int = 16, cmid: int = 32, cout: int = 32) -> GraphSpec:
    """conv3x3 + BN + ReLU -> conv1x1 + BN + ReLU -> maxpool 2x2 s2, fp32 (Table 1 row
    "Conv3x3 -> Conv1x1 -> MaxPooling")."""
    g = GraphSpec("single_chain", (cin, hw, hw), precision="fp32")
    x = g.cbr("c3", "input", cmid, 3, 1, 1)
    x = g.cbr("c1", x, cout, 1, 1, 0)
    g.pool("mp", x, "maxpool", 2, 2, 0)
    return g


def mobilenet_v1(hw: int = 224, width: float = 1.0, classes: int = 1000) -> GraphSpec:
    """Depthwise-separable stack: stem conv3x3 s2, 13 x (dw3x3 -> pw1x1), global avgpool, FC."""
    def ch(c):
        return max(8, int(c * width))
    g = GraphSpec("mobilenet_v1", (3, hw, hw))
    x = g.cbr("stem", "input", ch(32), 3, 2, 1, act="relu6")
    cfg = [(64, 1), (128, 2), (128, 1), (256, 2), (256, 1), (512, 2),
           (512, 1), (512, 1), (512, 1), (512, 1), (512, 1), (1024, 2), (1024, 1)]
    for i, (c, s) in enumerate(cfg, 1):
        cin = g.shapes[x][0]
        x = g.cbr(f"dw{i}", x, cin, 3, s, 1, groups=cin, act="relu6")
        x = g.cbr(f"pw{i}", x, ch(c), 1, 1, 0, act="relu6")
    x = g.gap("gap", x)
    g.fc("fc", x, classes)
    return g


def resnet18(hw: int = 224, base: int = 64, classes: int = 1000) -> GraphSpec:
    """conv7x7 s2 + maxpool 3x3 s2, four stages of two basic blocks, global avgpool, FC.
    Stage 1 keeps stride 1 with identity skips; stages 2-4 open with stride 2 and a 1x1
    stride-2 projection (+BN, no ReLU) on the skip."""
    g = GraphSpec("resnet18", (3, hw, hw))
    x = g.cbr("stem", "input", base, 7, 2, 3)
    x = g.pool("mp", x, "maxpool", 3, 2, 1)
    for si, c in enumerate([base, base * 2, base * 4, base * 8], 1):
        for bi in range(2):
            stride = 2 if (si > 1 and bi == 0) else 1
            n = f"s{si}b{bi}"
            y = g.cbr(n + ".c1", x, c, 3, stride, 1)
            y = g.cbr(n + ".c2", y, c, 3, 1, 1, act=None)
            skip = x
            if stride != 1 or g.shapes[x][0] != c:
                skip = g.cbr(n + ".proj", x, c, 1, stride, 0, act=None)
            y = g.add(n + ".add", y, skip)
            x = g.act(n + ".relu", y, "relu")
    x = g.gap("gap", x)
    g.fc("fc", x, classes)
    return g


def squeezenet11(hw: int = 224, classes: int = 1000, scale: int = 1) -> GraphSpec:
    """conv3x3 s2 (pad 0) + ReLU, maxpool, 8 fire modules with maxpools after fire 2 and 4,
    conv1x1 -> classes (no activation), global avgpool.  No BatchNorm: every conv has a bias."""
    g = GraphSpec("squeezenet11", (3, hw, hw))
    x = g.cbr("stem", "input", 64 // scale, 3, 2, 0, bn=False, bias=True)
    x = g.pool("mp0", x, "maxpool", 3, 2, 0)
    fires = [(16, 64), (16, 64), (32, 128), (32, 128), (48, 192), (48, 192), (64, 256), (64, 256)]
    for i, (s, e) in enumerate(fires, 1):
        s, e = s // scale, e // scale
        sq = g.cbr(f"f{i}.sq", x, s, 1, 1, 0, bn=False, bias=True)
        e1 = g.cbr(f"f{i}.e1", sq, e, 1, 1, 0, bn=False, bias=True)
        e3 = g.cbr(f"f{i}.e3", sq, e, 3, 1, 1, bn=False, bias=True)
        x = g.concat(f"f{i}.cat", [e1, e3])
        if i in (2, 4):
            x = g.pool(f"mp{i}", x, "maxpool", 3, 2, 0)
    x = g.cbr("cls", x, classes, 1, 1, 0, act=None, bn=False, bias=True)
    g.gap("gap", x)
    return g


def resnet50_stress(hw: int = 512, base: int = 64, blocks=(3, 4, 6, 3)) -> GraphSpec:
    """Bottleneck stages (1x1 reduce -> 3x3 -> 1x1 expand, residual add, ReLU), widths
    4*base*{1,2,4,8}; stride 2 on the 3x3 of the first block of stages 2-4; the first block of
    every stage has a 1x1 projection + BN on the skip; no classifier head."""
    g = GraphSpec("resnet50_stress", (3, hw, hw))
    x = g.cbr("stem", "input", base, 7, 2, 3)
    x = g.pool("mp", x, "maxpool", 3, 2, 1)
    for si, nb in enumerate(blocks, 1):
        mid = base * (2 ** (si - 1))
        out = mid * 4
        for bi in range(nb):
            stride = 2 if (si > 1 and bi == 0) else 1
            n = f"s{si}b{bi}"
            y = g.cbr(n + ".r", x, mid, 1, 1, 0)
            y = g.cbr(n + ".c3", y, mid, 3, stride, 1)
            y = g.cbr(n + ".e", y, out, 1, 1, 0, act=None)
            skip = x
            if bi == 0:
                skip = g.cbr(n + ".proj", x, out, 1, stride, 0, act=None)
            y = g.add(n + ".add", y, skip)
            x = g.act(n + ".relu", y, "relu")
    return g


# ------------------------------------------------------------------------------------------------
# The paper's operator micro-benchmarks (Table 4, Section 7.3)
# ------------------------------------------------------------------------------------------------
def operator_benchmark(name: str) -> GraphSpec:
    """One of the four operators of Table 4.  The table gives a feature map and a kernel per row and says which
    optimisation the row exercises (linking for the first two, split for the last two); pooling windows are not
    printed, and the first row's sizes are garbled ("224x224x24" with a kernel "3x3x3x224"): it is read as a
    224 x 224 x 3 image, a 3x3x3x24 kernel with stride 1 and padding 1 (a 224 x 224 x 24 map), then a 2 x 2
    stride-2 max pool; the average pool of the second row is the global average over the 7 x 7 map.  The fully
    connected row reads a 1 x 1 x 1536 map, flattened by a global average over its single pixel."""
    if name == "cbr_maxpool":
        g = GraphSpec("op_cbr_maxpool", (3, 224, 224))
        x = g.cbr("c", "input", 24, 3, 1, 1)
        g.pool("mp", x, "maxpool", 2, 2, 0)
    elif name == "cbr_avgpool":
        g = GraphSpec("op_cbr_avgpool", (1024, 7, 7))
        x = g.cbr("c", "input", 1024, 1, 1, 0)
        g.gap("ap", x)
    elif name == "fc":
        g = GraphSpec("op_fc", (1536, 1, 1))
        x = g.gap("flat", "input")
        g.fc("fc", x, 1000)
    elif name == "cbr":
        g = GraphSpec("op_cbr", (32, 112, 112))
        g.cbr("c", "input", 64, 1, 1, 0)
    else:
        raise ValueError(name)
    return g


OPERATOR_BENCHMARKS = ("cbr_maxpool", "cbr_avgpool", "fc", "cbr")


def config(i: int) -> Tuple[GraphSpec, List[int]]:
    """Workload i of the benchmark list with the batch sizes it is quoted at."""
    if i == 0:
        return single_chain(), [1]
    if i == 1:
        return mobilenet_v1(), [1, 32]
    if i == 2:
        return resnet18(), [1, 32]
    if i == 3:
        return squeezenet11(), [1, 32]
    if i == 4:
        return resnet50_stress(), [64]
    raise ValueError(i)
