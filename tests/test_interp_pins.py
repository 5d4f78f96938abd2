"""Pins for the graph interpreter of the CPU oracle (oracle/interp.py: run_graph).

Every whole-graph GPU parity check compares with run_graph, so run_graph itself is compared
here, bit for bit, with hand-written sequences of single-operator oracle calls (each of which has
its own pins in test_oracle_pins.py).  The graphs are built so that a mistake in the walk - stride
and pad exchanged, the wrong operand of an add, concat inputs in the wrong order, a dropped bias,
a pool given the wrong window - changes the result: every such pair of values differs.

The "original model" being walked is the operator list itself, one operator at a time
(Section 3 of the paper: the optimised model must be equivalent to it).
"""
import numpy as np
import pytest

import oracle as xo
from oracle import interp
from xenos_workloads import gen, graphs
from xenos_workloads.graphs import GraphSpec


def test_single_chain_equals_hand_written_sequence():
    spec = graphs.single_chain(hw=12)
    P = graphs.make_params(spec)
    x = graphs.make_input(spec, 2)
    y = xo.conv2d(x, P["c3"]["w"], None, 1, 1, 1)
    b = P["c3.bn"]
    y = xo.relu(xo.batchnorm(y, b["gamma"], b["beta"], b["mean"], b["var"], 1e-5))
    y = xo.conv2d(y, P["c1"]["w"], None, 1, 0, 1)
    b = P["c1.bn"]
    y = xo.relu(xo.batchnorm(y, b["gamma"], b["beta"], b["mean"], b["var"], 1e-5))
    y = xo.maxpool(y, 2, 2, 0)
    assert np.array_equal(interp.run_graph(spec, P, x), y)


def _mixed_graph():
    """One of each record kind, with parameters chosen so that no two arguments are interchangeable."""
    g = GraphSpec("mixed", (6, 13, 11), precision="fp32")
    a = g.conv("a", "input", 10, 5, stride=2, pad=1, bias=True)        # stride != pad, pad != k // 2
    a = g.bn("a.bn", a)
    a = g.act("a.relu6", a, "relu6")
    m = g.pool("m", a, "maxpool", 3, 1, 1)                             # k != stride, pad != 0, extent kept
    d = g.conv("d", a, 10, 3, stride=1, pad=1, groups=10)              # depthwise
    d = g.act("d.relu", d, "relu")
    s = g.add("s", m, d)
    s = g.act("s.relu", s, "relu")
    e = g.conv("e", s, 4, 1, bias=True)
    c = g.concat("c", [e, s])                                          # 4 + 10 channels: order matters
    p = g.pool("p", c, "avgpool", 2, 2, 0)
    v = g.gap("v", p)
    g.fc("f", v, 7, bias=True)
    return g


def _mixed_by_hand(P, x):
    t = {}
    b = P["a.bn"]
    t["a"] = xo.relu6(xo.batchnorm(xo.conv2d(x, P["a"]["w"], P["a"]["b"], 2, 1, 1), b["gamma"], b["beta"], b["mean"], b["var"], 1e-5))
    t["m"] = xo.maxpool(t["a"], 3, 1, 1)
    t["d"] = xo.relu(xo.conv2d(t["a"], P["d"]["w"], None, 1, 1, 10))
    t["s"] = xo.relu(xo.add(t["m"], t["d"]))
    t["e"] = xo.conv2d(t["s"], P["e"]["w"], P["e"]["b"], 1, 0, 1)
    t["c"] = xo.concat([t["e"], t["s"]])
    t["p"] = xo.avgpool(t["c"], 2, 2, 0)
    t["v"] = xo.global_avgpool(t["p"])
    t["f"] = xo.fc(t["v"], P["f"]["w"], P["f"]["b"])
    return t


def test_mixed_graph_equals_hand_written_sequence_bit_exact():
    spec = _mixed_graph()
    P = graphs.make_params(spec)
    x = graphs.make_input(spec, 3)
    t = _mixed_by_hand(P, x)
    got = interp.run_graph(spec, P, x, keep=True)
    for name, mine in [("a.relu6", "a"), ("m", "m"), ("d.relu", "d"), ("s.relu", "s"), ("e", "e"), ("c", "c"), ("p", "p"),
                       ("v", "v"), ("f", "f")]:
        assert got[name].shape == t[mine].shape, name
        assert np.array_equal(got[name], t[mine]), name
    assert np.array_equal(interp.run_graph(spec, P, x), t["f"])


def test_the_hand_written_sequence_would_notice_swapped_arguments():
    """The pin above has teeth: each plausible slip in the walk changes some tensor of this graph."""
    spec = _mixed_graph()
    P = graphs.make_params(spec)
    x = graphs.make_input(spec, 1)
    t = _mixed_by_hand(P, x)
    # stride and pad exchanged in the strided convolution: another extent altogether
    assert xo.conv2d(x, P["a"]["w"], P["a"]["b"], 1, 2, 1).shape != t["a"].shape
    # pool window arguments exchanged
    assert not np.array_equal(xo.maxpool(t["a"], 3, 1, 1), xo.maxpool(t["a"], 1, 1, 0))
    # concat in the wrong order
    assert not np.array_equal(t["c"], xo.concat([t["s"], t["e"]]))
    # a dropped bias
    assert not np.array_equal(t["e"], xo.conv2d(t["s"], P["e"]["w"], None, 1, 0, 1))
    assert not np.array_equal(t["f"], xo.fc(t["v"], P["f"]["w"], None))
    # relu in place of relu6 (values above 6 exist after the first convolution's batch norm scale)
    b = P["a.bn"]
    pre = xo.batchnorm(xo.conv2d(x * 8.0, P["a"]["w"], P["a"]["b"], 2, 1, 1), b["gamma"], b["beta"], b["mean"], b["var"], 1e-5)
    assert pre.max() > 6.0 and not np.array_equal(xo.relu(pre), xo.relu6(pre))


def test_add_reads_both_operands_and_in_either_order():
    g = GraphSpec("addg", (4, 5, 5), precision="fp32")
    a = g.conv("a", "input", 4, 1)
    b = g.conv("b", "input", 4, 3, 1, 1)
    g.add("s", b, a)
    P = graphs.make_params(g)
    x = graphs.make_input(g, 2)
    ya, yb = xo.conv2d(x, P["a"]["w"], None, 1, 0, 1), xo.conv2d(x, P["b"]["w"], None, 1, 1, 1)
    assert np.array_equal(interp.run_graph(g, P, x), xo.add(yb, ya))
    assert not np.array_equal(xo.add(yb, ya), xo.add(ya, ya))


def test_bf16_emulation_rounds_stored_tensors_only():
    """The diagnostic mode rounds the input and the end of every fused group (conv [+bn] [+act], add [+act]),
    and nothing inside a group: the same rounding points the device has."""
    g = GraphSpec("emu", (8, 6, 6))
    a = g.cbr("a", "input", 8, 3, 1, 1, act="relu")
    b = g.cbr("b", a, 8, 1, act=None)
    s = g.add("s", b, a)
    g.act("s.relu", s, "relu")
    P = graphs.make_params(g)
    x = graphs.make_input(g, 2)
    r = xo.round_bf16
    bn = lambda y, q: xo.batchnorm(y, q["gamma"], q["beta"], q["mean"], q["var"], 1e-5)
    ya = r(xo.relu(bn(xo.conv2d(r(x), P["a"]["w"], None, 1, 1, 1), P["a.bn"])))
    yb = bn(xo.conv2d(ya, P["b"]["w"], None, 1, 0, 1), P["b.bn"])          # feeds the add: not stored, not rounded
    ys = r(xo.relu(xo.add(yb, ya)))
    assert np.array_equal(interp.run_graph(g, P, x, bf16_emulate=True), ys)


@pytest.mark.parametrize("tile", [(1, 1), (2, 3), (7, 7)])
def test_avgpool_stage_of_the_tiled_chain_equals_the_plain_average_pool(tile):
    """conv3x3 -> conv1x1 -> average pool 2x2, tile by tile, against one operator at a time (Table 1, the
    ConvX -> ConvY -> AvgPooling row)."""
    rng_seed = gen.DEFAULT_SEED + 5
    x = gen.uniform(rng_seed, 0, (2, 5, 14, 14), -1.0, 1.0)
    w1 = gen.normal(rng_seed, 1, (6, 5, 3, 3), 0.0, 0.3)
    w2 = gen.normal(rng_seed, 2, (4, 6, 1, 1), 0.0, 0.5)
    b2 = gen.uniform(rng_seed, 3, (4,), -0.1, 0.1)
    plain = xo.avgpool(xo.conv2d(xo.relu(xo.conv2d(x, w1, None, 1, 1, 1)), w2, b2, 1, 0, 1), 2, 2, 0)
    stages = [dict(kind="conv", w=w1, stride=1, pad=1, act="relu"), dict(kind="conv", w=w2, bias=b2),
              dict(kind="avgpool", k=2, stride=2, pad=0)]
    tiled = xo.chain_tiled(x, stages, tile[0], tile[1])
    assert np.array_equal(tiled, plain)
    # and the average itself against the mean of each window, in float64
    ref = xo.conv2d(xo.relu(xo.conv2d(x, w1, None, 1, 1, 1)), w2, b2, 1, 0, 1).astype(np.float64)
    ref = ref.reshape(2, 4, 7, 2, 7, 2).mean(axis=(3, 5))
    assert np.abs(plain - ref).max() <= 1e-6


def test_matrix_operators_equal_hand_written_sequence():
    """x.matmul (with and without bias), x.transpose, x.split, x.mul and x.mac walked by run_graph against the same
    operators called by hand; the operands of mac and the parts of the split are all different."""
    g = GraphSpec("matrix", (8, 6, 1), precision="fp32")
    q = g.matmul("q", "input", 12, bias=True)
    k = g.matmul("k", "input", 12)
    lo = g.split("lo", q, 0, 4)
    hi = g.split("hi", q, 8, 4)
    mid = g.split("mid", k, 4, 4)
    m = g.mul("m", lo, hi)
    a = g.mac("a", m, mid, lo)
    g.transpose("t", a)
    P = graphs.make_params(g)
    x = graphs.make_input(g, 3)
    qv = xo.matmul(x, P["q"]["w"], P["q"]["b"])
    kv = xo.matmul(x, P["k"]["w"], None)
    lov, hiv, midv = xo.split_part(qv, 0, 4), xo.split_part(qv, 8, 4), xo.split_part(kv, 4, 4)
    want = xo.transpose(xo.mac(xo.mul(lov, hiv), midv, lov))
    got = interp.run_graph(g, P, x)
    assert got.shape == (3, 6, 4, 1) and np.array_equal(got, want)
