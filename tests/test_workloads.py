"""Workload graph records: shapes, MAC counts and end-to-end oracle evaluation."""
import os

import numpy as np
import pytest

import oracle as xo
from oracle import interp
from xenos_workloads import graphs

GOLD = os.path.join(os.path.dirname(__file__), "golden", "workload_anchors.txt")


def _anchors():
    rows = []
    for line in open(GOLD):
        if line.strip() and not line.startswith("#"):
            name, hw, macs, shape, nconv, nops = line.split()
            rows.append((name, int(hw), int(macs), tuple(int(v) for v in shape.split(",")), int(nconv), int(nops)))
    return rows


@pytest.mark.parametrize("row", _anchors(), ids=lambda r: r[0])
def test_graph_matches_anchor(row):
    name, hw, macs, shape, nconv, nops = row
    spec = getattr(graphs, name)()
    assert spec.in_shape[1] == hw
    assert spec.macs() == macs
    assert spec.shapes[spec.output] == shape
    assert sum(o["kind"] == "conv" for o in spec.ops) == nconv
    assert len(spec.ops) == nops


def test_squeezenet_pool_extents_do_not_depend_on_rounding_mode():
    spec = graphs.squeezenet11()
    assert spec.shapes["stem.relu"][1:] == (111, 111)
    assert spec.shapes["mp0"][1:] == (55, 55)
    assert spec.shapes["mp2"][1:] == (27, 27)
    assert spec.shapes["mp4"][1:] == (13, 13)


def test_small_graphs_run_and_bf16_emulation_stays_close():
    for spec in (graphs.mobilenet_v1(hw=32, width=0.25, classes=10), graphs.resnet18(hw=32, base=8, classes=10),
                 graphs.squeezenet11(hw=47, classes=10, scale=4), graphs.resnet50_stress(hw=32, base=8, blocks=(1, 1, 1, 1))):
        P = graphs.make_params(spec)
        x = graphs.make_input(spec, 2)
        y = interp.run_graph(spec, P, x)
        assert y.shape == (2,) + spec.shapes[spec.output]
        assert np.isfinite(y).all()
        # images are independent: evaluating image 1 alone gives the same bits
        y1 = interp.run_graph(spec, P, x[1:2])
        assert np.array_equal(y1[0], y[1])
        yb = interp.run_graph(spec, P, x, bf16_emulate=True)
        assert np.abs(yb - y).max() <= 2e-2 * np.abs(y).max()
