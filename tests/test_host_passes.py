"""Host logic of the C-ABI library, no GPU needed: exported symbols, the call-order state machine,
error codes, Conv-Bn-Relu pre-fusion, Table 1 pattern matching, split plans (exact covers,
halos, determinism) and the workspace layout."""
import ctypes
import itertools
import os
import re

import numpy as np
import pytest

from paper_2302_00282_b200 import binding as xb
from xenos_workloads import graphs
from xenos_workloads.feed import graph_from_spec
from xenos_workloads.graphs import GraphSpec

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = os.path.join(os.path.dirname(__file__), "golden", "link_patterns.txt")


def compiled(spec, batch=2, linked=True, splits=(), links=None, hw=None, nhwc=False):
    P = graphs.make_params(spec)
    g, ids = graph_from_spec(spec, P, hw=hw, in_dtype=xb.DTYPE_BF16 if nhwc else None, in_layout=xb.LAYOUT_NHWC if nhwc else None)
    if links is not None:
        for ch in links:
            g.link([ids[n] for n in ch])
    elif linked:
        g.link()
    for name, kw in splits:
        g.split(ids[name], **kw)
    g.compile(batch, xb.PRECISION_FP32_CUDA_CORE if spec.precision == "fp32" else xb.PRECISION_BF16_TENSOR)
    return g, ids


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "xenos.h")).read()
    declared = sorted(set(re.findall(r"\b(xenos_(?:graph_\w+|last_error))\s*\(", hdr)))
    assert declared and sorted(xb.EXPORTS) == declared
    L = xb.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_state_machine_and_argument_errors():
    g = xb.Graph()
    with pytest.raises(xb.XenosError) as e:
        g.compile(1, xb.PRECISION_BF16_TENSOR)
    assert e.value.code == xb.E_INVALID                      # no input yet
    x = g.add_input(xb.DTYPE_F32, xb.LAYOUT_NCHW, 4, 8, 8)
    w = np.ones((4, 4, 3, 3), np.float32)
    with pytest.raises(xb.XenosError) as e:
        g.add_op(xb.OP_CONV, [x], cout=4, k=9, stride=1, pad=0, weight=np.ones((4, 4, 9, 9), np.float32))
    assert e.value.code == xb.E_SHAPE                        # kernel larger than the input
    with pytest.raises(xb.XenosError) as e:
        g.add_op(xb.OP_CONV, [x], cout=4, k=3, weight=None)
    assert e.value.code == xb.E_INVALID
    with pytest.raises(xb.XenosError) as e:
        g.add_op(xb.OP_CONV, [x], cout=4, k=3, groups=2, weight=np.ones((4, 2, 3, 3), np.float32))
    assert e.value.code == xb.E_UNSUPPORTED                  # grouped but not depthwise
    with pytest.raises(xb.XenosError) as e:
        g.add_op(42, [x])
    assert e.value.code == xb.E_UNSUPPORTED                  # x.mul / x.mac / ... are not implemented
    with pytest.raises(xb.XenosError) as e:
        g.add_op(xb.OP_CONV, [99], cout=4, k=3, weight=w)
    assert e.value.code == xb.E_INVALID
    y = g.add_op(xb.OP_CONV, [x], cout=4, k=3, stride=1, pad=1, weight=w)
    z = g.add_op(xb.OP_POOL_MAX, [y], k=2, stride=2)
    with pytest.raises(xb.XenosError) as e:
        g.add_op(xb.OP_ADD, [y, z])
    assert e.value.code == xb.E_SHAPE
    with pytest.raises(xb.XenosError) as e:
        g.link([y])
    assert e.value.code == xb.E_NOT_LINKABLE
    with pytest.raises(xb.XenosError) as e:
        g.link([z, y])                                       # not producer -> consumer
    assert e.value.code == xb.E_NOT_LINKABLE
    with pytest.raises(xb.XenosError) as e:
        g.split(y, parts_k=-2)
    assert e.value.code == xb.E_BAD_SPLIT
    for call in (lambda: g.bind(256, 256), lambda: g.run(1, [1], [1]), lambda: g.plan(), lambda: g.status()):
        with pytest.raises(xb.XenosError) as e:
            call()
        assert e.value.code == xb.E_STATE
    g.mark_output(z, xb.DTYPE_F32, xb.LAYOUT_NCHW)
    with pytest.raises(xb.XenosError) as e:
        g.mark_output(z, xb.DTYPE_F32, xb.LAYOUT_NCHW)
    assert e.value.code == xb.E_INVALID
    n = g.compile(3, xb.PRECISION_FP32_CUDA_CORE)
    assert n > 0
    for call in (lambda: g.add_input(0, 0, 1, 1, 1), lambda: g.link(), lambda: g.split(-1),
                 lambda: g.compile(3, 0), lambda: g.run(1, [1], [1])):
        with pytest.raises(xb.XenosError) as e:
            call()
        assert e.value.code == xb.E_STATE
    with pytest.raises(xb.XenosError) as e:
        g.bind(0, n)
    assert e.value.code == xb.E_WORKSPACE
    with pytest.raises(xb.XenosError) as e:
        g.bind(4096 + 8, n)                                  # misaligned
    assert e.value.code == xb.E_WORKSPACE
    with pytest.raises(xb.XenosError) as e:
        g.bind(4096, n - 1)
    assert e.value.code == xb.E_WORKSPACE
    g.destroy()


def test_bind_fails_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    g, _ = compiled(graphs.single_chain(), 1)
    n = g.plan()["workspace_bytes"]
    with pytest.raises(xb.XenosError) as e:
        g.bind(1 << 20, max(n, 256))
    assert e.value.code == xb.E_CUDA


def test_split_search_needs_a_device_and_the_build_state():
    """The PROFILING step of the search runs on the GPU: without one the call fails loudly and leaves the graph as
    it was; after compile the call is out of order."""
    spec = graphs.mobilenet_v1(hw=32, width=0.25, classes=8)
    P = graphs.make_params(spec)
    g, _ = graph_from_spec(spec, P)
    g.link()
    with pytest.raises(xb.XenosError) as e:
        g.search_split(2, xb.PRECISION_BF16_TENSOR, 256, 1 << 30, [256], [256])
    assert e.value.code in (xb.E_CUDA, xb.E_WORKSPACE)
    with pytest.raises(xb.XenosError) as e:
        g.search_split(2, xb.PRECISION_BF16_TENSOR, 0, 1 << 30, [256], [256])
    assert e.value.code == xb.E_WORKSPACE
    g.compile(2, xb.PRECISION_BF16_TENSOR)
    with pytest.raises(xb.XenosError) as e:
        g.search_split(2, xb.PRECISION_BF16_TENSOR, 256, 1 << 30, [256], [256])
    assert e.value.code == xb.E_STATE


def test_prefusion_folds_bn_and_activation():
    spec = graphs.single_chain()
    g, _ = compiled(spec, 1, linked=False)
    pl = g.plan()
    assert [n["kind"] for n in pl["nodes"]] == ["conv", "conv", "maxpool"]
    assert [len(n["user_ops"]) for n in pl["nodes"]] == [3, 3, 1]
    assert [n["act"] for n in pl["nodes"]] == [1, 1, 0]
    assert len(pl["chains"]) == 3 and all(c["kind"] == "single" for c in pl["chains"])


def test_standalone_bn_or_activation_is_rejected():
    g = xb.Graph()
    x = g.add_input(xb.DTYPE_F32, xb.LAYOUT_NCHW, 4, 8, 8)
    p = g.add_op(xb.OP_POOL_MAX, [x], k=2, stride=2)
    r = g.add_op(xb.OP_RELU, [p])
    g.mark_output(r, xb.DTYPE_F32, xb.LAYOUT_NCHW)
    with pytest.raises(xb.XenosError) as e:
        g.compile(1, xb.PRECISION_FP32_CUDA_CORE)
    assert e.value.code == xb.E_UNSUPPORTED


def _gold_counts():
    out = {}
    for line in open(GOLD):
        if line.strip() and not line.startswith("#"):
            name, pat, cnt = line.split()
            out.setdefault(name, {})[pat] = int(cnt)
    return out


def _classify(chain, nodes):
    kinds = [nodes[i]["kind"] for i in chain["nodes"]]
    if chain["kind"] == "conv_conv_pool":
        return "conv-conv-pool"
    if chain["kind"] == "dw_pw":
        return "dw-pw"
    if chain["kind"] == "expand_concat":
        return "fire"
    if chain["kind"] == "conv_conv":      # the deeper form of a row: the first convolution's result stays on chip
        return "fire" if "concat" in kinds else ("shortcut" if "add" in kinds else "conv-conv")
    if chain["kind"] == "conv_tail":
        if "add" in kinds:
            return "shortcut"
        return "conv-pool" if "maxpool" in kinds else "conv-gap"
    return None


@pytest.mark.parametrize("name", ["single_chain", "mobilenet_v1", "resnet18", "squeezenet11", "resnet50_stress"])
def test_table1_patterns_are_found(name):
    spec = getattr(graphs, name)()
    g, _ = compiled(spec, 1)
    pl = g.plan()
    got = {}
    for c in pl["chains"]:
        k = _classify(c, pl["nodes"])
        if k:
            got[k] = got.get(k, 0) + 1
    want = _gold_counts()[name]
    on_chip = want.pop("on-chip", None)
    if on_chip is not None:
        assert sum(c["kind"] == "conv_conv" for c in pl["chains"]) == on_chip
    if name == "mobilenet_v1":        # the last dw -> pw chain also absorbs the global average
        want = {"dw-pw": 13}
        assert sum("gap" in [pl["nodes"][i]["kind"] for i in c["nodes"]] for c in pl["chains"]) == 1
    if name == "squeezenet11":        # 13x13 = 169 rows: the classifier -> gap chain averages over two 128-row tiles
        L = [l for l in pl["launches"] if l.get("gap_parts", 1) > 1]
        assert len(L) == 1 and L[0]["gap_parts"] == 2 and L[0]["m_tiles"] == 2 * pl["max_batch"]
    assert got == want
    # every node is in exactly one chain; chains run after their producers
    seen = sorted(i for c in pl["chains"] for i in c["nodes"])
    assert seen == list(range(len(pl["nodes"])))
    produced = set(t["id"] for t in pl["tensors"] if t["external"])
    for L in pl["launches"]:
        for t in (L["in0"], L["in1"], L["skip"]):
            assert t < 0 or t in produced, (L["id"], t)
        produced.add(L["out"])


def test_producer_with_two_unrelated_consumers_is_not_linked():
    g = GraphSpec("fork", (16, 12, 12))
    a = g.cbr("a", "input", 16, 3, 1, 1)
    p = g.pool("p", a, "maxpool", 2, 2)
    q = g.cbr("q", a, 16, 1)          # second consumer of a
    g.pool("q.p", q, "maxpool", 2, 2)
    g.output = "p"
    gg, _ = compiled(g, 1)
    pl = gg.plan()
    chain_of = {n["id"]: n["chain"] for n in pl["nodes"]}
    assert pl["chains"][chain_of[0]]["kind"] == "single"     # a -> {p, q}: a stays alone


def test_explicit_link_requests():
    spec = graphs.mobilenet_v1(hw=32, width=0.25, classes=8)
    g, _ = compiled(spec, 1, links=[["dw1", "pw1"], ["dw13", "pw13", "gap"]])
    pl = g.plan()
    linked = [c for c in pl["chains"] if c["kind"] != "single"]
    assert len(linked) == 2 and [len(c["nodes"]) for c in linked] == [2, 3]
    with pytest.raises(xb.XenosError) as e:
        compiled(spec, 1, links=[["pw1", "dw2"]])            # adjacent, but no pattern with a kernel
    assert e.value.code == xb.E_NOT_LINKABLE
    with pytest.raises(xb.XenosError) as e:
        compiled(spec, 1, links=[["dw1", "pw1"], ["dw1", "pw1"]])
    assert e.value.code == xb.E_NOT_LINKABLE


def test_plans_are_deterministic():
    for spec in (graphs.single_chain(), graphs.resnet18(hw=64, base=16, classes=8)):
        a, _ = compiled(spec, 4)
        b, _ = compiled(spec, 4)
        assert a.plan_text() == b.plan_text()


@pytest.mark.parametrize("split", [dict(), dict(parts_outc=4, parts_h=2, parts_w=1), dict(parts_outc=2, parts_h=4, parts_w=8),
                                   dict(parts_h=16, parts_w=16), dict(parts_outc=32)])
def test_fp32_chain_split_is_an_exact_cover_with_correct_halo(split):
    spec = graphs.single_chain()
    g, _ = compiled(spec, 1, splits=[("mp", split)] if split else ())
    L = g.plan()["launches"][0]
    assert L["kind"] == "f32_conv_conv_pool"
    PP = PQ = 16
    if split.get("parts_outc"):
        assert L["parts_outc"] == split["parts_outc"]
    if split.get("parts_h"):
        assert L["tiles_h"] == split["parts_h"] and L["tiles_w"] == split.get("parts_w", L["tiles_w"])
    cover = np.zeros((32, PP, PQ), int)
    kper = 32 // L["parts_outc"]
    for part, ty, tx in itertools.product(range(L["parts_outc"]), range(L["tiles_h"]), range(L["tiles_w"])):
        y0, x0 = ty * L["tile_h"], tx * L["tile_w"]
        cover[part * kper:(part + 1) * kper, y0:min(PP, y0 + L["tile_h"]), x0:min(PQ, x0 + L["tile_w"])] += 1
    assert (cover == 1).all()                                 # disjoint and complete
    assert L["grid"] == L["parts_outc"] * L["tiles_h"] * L["tiles_w"]
    # halo: rows / columns of the first conv's output a full tile reads (pool 2x2 s2 over a 1x1 conv)
    assert (L["halo_h"], L["halo_w"]) == (2 * L["tile_h"], 2 * L["tile_w"])


def test_bad_splits_are_rejected():
    spec = graphs.single_chain()
    for kw in (dict(parts_outc=5), dict(parts_h=17), dict(parts_w=64), dict(parts_outc=64)):
        with pytest.raises(xb.XenosError) as e:
            compiled(spec, 1, splits=[("mp", kw)])
        assert e.value.code == xb.E_BAD_SPLIT, kw
    m = graphs.mobilenet_v1(hw=32, width=0.25, classes=8)
    with pytest.raises(xb.XenosError) as e:
        compiled(m, 1, splits=[("pw1.relu6", dict(parts_h=2))])
    assert e.value.code == xb.E_BAD_SPLIT


def test_gemm_split_prefers_output_channels_until_units_are_busy():
    """Section 4.2.1: kernels are dealt to the units first; rows / columns follow."""
    spec = graphs.mobilenet_v1()
    for batch in (1, 32):
        g, _ = compiled(spec, batch)
        for L in g.plan()["launches"]:
            if L["kind"] != "gemm":
                continue
            assert L["tile_n"] % 16 == 0 and 16 <= L["tile_n"] <= 256
            cols = L["tile_n"] * L["n_acc"]                   # columns of a CTA's tile
            assert L["npad"] == cols * L["n_tiles"] and (L["n_tiles"] - 1) * cols < L["K"] <= L["npad"]
            assert L["grid"] == min(148, L["m_tiles"] * L["n_tiles"] * L["ksplit"])     # one persistent CTA per unit
            if L["n_tiles"] * L["n_acc"] > -(-L["K"] // 256):  # split finer than the 256-wide maximum
                assert L["m_tiles"] * (L["n_tiles"] // 2) < 148   # ... only because units would idle otherwise
                if L["a0"] == "dw":
                    # a linked depthwise stage is recomputed per channel tile: narrow tiles only while at least three
                    # quarters of the units would otherwise idle
                    assert L["tile_n"] >= 128 or L["m_tiles"] * -(-L["K"] // 256) * 4 <= 148
            assert L["tmem_cols"] >= 2 * L["tile_n"] and 1 <= L["stages"] <= 6
            assert L["smem_bytes"] <= 227 * 1024
            if L["a0"] == "dw":
                assert L["ni"] * L["patch_rh"] * L["patch_rw"] <= 128 and L["hstages"] >= 2
    hw = xb.HwInfo(16, 227 * 1024, 512, 1 << 20)
    g2, _ = compiled(spec, 1, hw=hw)
    assert g2.plan()["hw"]["sm_count"] == 16


def _unit(build, cin, hw):
    g = GraphSpec("unit", (cin, hw, hw))
    build(g)
    return g


@pytest.mark.parametrize("parts_k", [2, 3, 4, 6, 9, 18, 36])
def test_reduction_split_is_an_ascending_exact_cover_of_the_k_blocks(parts_k):
    """Section 4.2.2: the reduction (C, R, S) is cut last and needs an additional reduction.  Here: chunks of
    64-element K blocks, equal size, ascending, disjoint, complete."""
    spec = _unit(lambda g: g.cbr("c", "input", 48, 3, 1, 1), 256, 6)        # K = 256 * 9 = 36 blocks
    g, _ = compiled(spec, 2, linked=False, splits=[("c", dict(parts_k=parts_k))], nhwc=True)
    L = g.plan()["launches"][0]
    assert L["kblocks"] == 36 and L["ksplit"] == parts_k
    chunks = [(s * L["kb_per"], min(L["kblocks"], (s + 1) * L["kb_per"])) for s in range(L["ksplit"])]
    assert chunks[0][0] == 0 and chunks[-1][1] == L["kblocks"]
    assert all(a < b for a, b in chunks) and all(chunks[i][1] == chunks[i + 1][0] for i in range(len(chunks) - 1))
    assert L["grid"] == min(148, L["m_tiles"] * L["n_tiles"] * parts_k)


def test_reduction_split_requests_that_cannot_be_met():
    spec = _unit(lambda g: g.cbr("c", "input", 48, 3, 1, 1), 256, 6)
    for pk, code in ((37, xb.E_BAD_SPLIT), (7, xb.E_BAD_SPLIT), (10, xb.E_BAD_SPLIT)):     # 36 blocks: 7 -> 6 chunks of 6, 10 -> 9 of 4
        with pytest.raises(xb.XenosError) as e:
            compiled(spec, 2, linked=False, splits=[("c", dict(parts_k=pk))], nhwc=True)
        assert e.value.code == code, pk
    m = graphs.mobilenet_v1(hw=32, width=0.25, classes=8)
    with pytest.raises(xb.XenosError) as e:
        compiled(m, 1, splits=[("stem.relu6", dict(parts_k=2))])       # a convolution that reads the image
    assert e.value.code == xb.E_UNSUPPORTED
    with pytest.raises(xb.XenosError) as e:
        compiled(m, 1, splits=[("pw1.relu6", dict(parts_k=2))])        # depthwise -> pointwise with one K block
    assert e.value.code == xb.E_BAD_SPLIT
    with pytest.raises(xb.XenosError) as e:
        compiled(graphs.single_chain(), 1, splits=[("mp", dict(parts_k=2))])     # fp32 CUDA-core chain
    assert e.value.code == xb.E_UNSUPPORTED


def test_reduction_split_is_automatic_only_where_units_would_idle():
    spec = graphs.mobilenet_v1()
    g, _ = compiled(spec, 32)
    L = g.plan()["launches"]
    assert [l.get("ksplit", 1) for l in L[:-1]] == [1] * (len(L) - 1)
    fc = L[-1]
    assert fc["ksplit"] >= 2 and fc["m_tiles"] * fc["n_tiles"] * fc["ksplit"] <= 148 and fc["kb_per"] >= 2 and not fc["fc_small"]
    # up to 8 vectors the fc is one pass over its weights on the CUDA cores: no tiles to cut
    fc8 = compiled(spec, 8)[0].plan()["launches"][-1]
    assert fc8["fc_small"] == 1 and fc8["ksplit"] == 1
    # a depthwise -> pointwise chain is cut on request only
    g1, ids = compiled(spec, 1, splits=[("pw7.relu6", dict(parts_k=8))])
    L1 = g1.plan()["launches"]
    assert [l.get("ksplit", 1) for l in L1 if l.get("a0") == "dw"].count(8) == 1
    assert all(l["ksplit"] == 1 for l in L1 if l.get("a0") == "stem" or l.get("epi") in (1, 2))


def test_user_outc_split_sets_tiles():
    spec = graphs.mobilenet_v1()
    g, ids = compiled(spec, 32, splits=[("pw7.relu6", dict(parts_outc=4))])
    pl = g.plan()
    node = [n for n in pl["nodes"] if n["out"] == ids["pw7.relu6"]][0]
    L = pl["launches"][pl["chains"][node["chain"]]["launches"][0]]
    assert (L["n_tiles"], L["tile_n"]) == (4, 128)


def test_pool_patch_tiles_cover_pool_output():
    spec = graphs.resnet18()
    g, _ = compiled(spec, 2)
    L = [l for l in g.plan()["launches"] if l["kind"] == "gemm" and l["epi"] == 2][0]
    assert L["patch_rh"] == (L["patch_th"] - 1) * 2 + 3 and L["patch_rw"] == (L["patch_tw"] - 1) * 2 + 3
    assert L["patch_rh"] * L["patch_rw"] <= 128
    assert L["tiles_y"] * L["patch_th"] >= 56 > (L["tiles_y"] - 1) * L["patch_th"]
    assert L["tiles_x"] * L["patch_tw"] >= 56 > (L["tiles_x"] - 1) * L["patch_tw"]
    assert L["m_tiles"] == 2 * L["tiles_y"] * L["tiles_x"]


@pytest.mark.parametrize("name,kw", [("mobilenet_v1", {}), ("resnet18", {}), ("squeezenet11", {}),
                                     ("resnet50_stress", dict(hw=128))])
@pytest.mark.parametrize("linked", [True, False])
def test_workspace_tensors_never_overlap_while_live(name, kw, linked):
    spec = getattr(graphs, name)(**kw)
    g, _ = compiled(spec, 2, linked=linked)
    pl = g.plan()
    ts = [t for t in pl["tensors"] if not t["external"]]
    for a, b in itertools.combinations(ts, 2):
        live = not (a["last"] < b["first"] or b["last"] < a["first"])
        mem = not (a["off"] + a["bytes"] <= b["off"] or b["off"] + b["bytes"] <= a["off"])
        assert not (live and mem), (a, b)
    for t in ts:
        assert t["off"] >= pl["param_bytes"] and t["off"] + t["bytes"] <= pl["workspace_bytes"] and t["off"] % 256 == 0
    # linking removes intermediates from memory
    if linked:
        gu, _ = compiled(spec, 2, linked=False)
        assert pl["bytes_linked"] < gu.plan()["bytes_linked"]
        assert len(pl["launches"]) < len(gu.plan()["launches"])


def test_modelled_work_matches_shapes():
    spec = graphs.mobilenet_v1()
    g, _ = compiled(spec, 32)
    pl = g.plan()
    assert pl["flops"] == 2 * 32 * spec.macs()
    # depthwise-separable chains dominate the saving: linked bytes are well below unlinked ones
    assert pl["bytes_linked"] < 0.7 * pl["bytes_unlinked"]


# ---- the remaining operators of Table 3 and the MatmulX -> MatmulY link ---------------------------------
def _matrix_graph(act_between=None, n1=64, n2=32, bias=True):
    g = GraphSpec("mm", (64, 16, 1))
    a = g.matmul("m1", "input", n1, bias=bias)
    if act_between:
        a = g.act("m1." + act_between, a, act_between)
    g.matmul("m2", a, n2, bias=bias)
    return g


def test_matmul_matmul_is_linked_by_multiplying_the_constants():
    g, _ = compiled(_matrix_graph(), 4, nhwc=True)
    pl = g.plan()
    assert [c["kind"] for c in pl["chains"]] == ["matmul_matmul"] and len(pl["launches"]) == 1
    assert "MatmulX -> MatmulY" in pl["chains"][0]["pattern"]
    L = pl["launches"][0]
    assert (L["C"], L["K"]) == (64, 32) and L["flops"] == 2 * 4 * 16 * 64 * 32
    # an activation between the two products, or a merged product with more multiplications, is not linked
    g2, _ = compiled(_matrix_graph(act_between="relu"), 4, nhwc=True)
    assert len(g2.plan()["launches"]) == 2
    g3, _ = compiled(_matrix_graph(n1=8, n2=256), 4, nhwc=True)          # 64 * 256 > 64 * 8 + 8 * 256
    assert len(g3.plan()["launches"]) == 2
    # unlinked: two launches
    g4, _ = compiled(_matrix_graph(), 4, linked=False, nhwc=True)
    assert len(g4.plan()["launches"]) == 2


def test_matrix_operator_shapes_and_errors():
    g = xb.Graph()
    x = g.add_input(xb.DTYPE_BF16, xb.LAYOUT_NHWC, 16, 8, 1)
    w = np.ones((16, 24), np.float32)
    m = g.add_op(xb.OP_MATMUL, [x], cout=24, k=1, weight=w)
    t = g.add_op(xb.OP_TRANSPOSE, [m])
    s = g.add_op(xb.OP_SPLIT, [m], cout=8, pad=16)
    g.add_op(xb.OP_MUL, [s, s])
    g.add_op(xb.OP_MAC, [s, s, s])
    for call, code in ((lambda: g.add_op(xb.OP_MATMUL, [x, m], cout=24, k=1, weight=w), xb.E_UNSUPPORTED),   # two run-time operands
                       (lambda: g.add_op(xb.OP_SPLIT, [m], cout=16, pad=16), xb.E_SHAPE),                  # leaves the input
                       (lambda: g.add_op(xb.OP_MUL, [s, m]), xb.E_SHAPE),
                       (lambda: g.add_op(xb.OP_MAC, [s, s]), xb.E_INVALID),
                       (lambda: g.add_op(xb.OP_MATMUL, [x], cout=24, k=1), xb.E_INVALID)):                  # no constant
        with pytest.raises(xb.XenosError) as e:
            call()
        assert e.value.code == code
    y = g.add_input(xb.DTYPE_BF16, xb.LAYOUT_NHWC, 16, 8, 2)
    with pytest.raises(xb.XenosError) as e:
        g.add_op(xb.OP_TRANSPOSE, [y])                       # width 2: not a matrix
    assert e.value.code == xb.E_SHAPE
    g.mark_output(t, xb.DTYPE_BF16, xb.LAYOUT_NHWC)
    g.compile(2, xb.PRECISION_BF16_TENSOR)
    pl = g.plan()
    tt = [n for n in pl["nodes"] if n["kind"] == "transpose"][0]
    assert tt["cin"] == 24 and tt["cout"] == 8               # (24 columns, 8 rows) -> (8 columns, 24 rows)


def test_stress_graph_keeps_the_bottleneck_tails_on_chip():
    """ConvX -> ConvY (3x3 -> 1x1 expand) + identity shortcut in one kernel for the blocks of stages 1-3 that have no
    shortcut convolution; the blocks that have one keep the shortcut row's link; stage 4 (512 middle channels) does
    not fit the accumulators."""
    spec = graphs.resnet50_stress()
    g, _ = compiled(spec, 64)
    pl = g.plan()
    cc = [c for c in pl["chains"] if c["kind"] == "conv_conv"]
    assert len(cc) == _gold_counts()["resnet50_stress"]["on-chip"] and len(pl["launches"]) == 39
    for c in cc:
        kinds = [pl["nodes"][i]["kind"] for i in c["nodes"]]
        L = pl["launches"][c["launches"][0]]
        assert kinds == ["conv", "conv", "add"] and L["kind"] == "gemm2" and L["k"] == 3 and L["k2"] == 1 and L["skip"] >= 0
        assert L["cmid"] in (64, 128, 256) and L["patch_rh"] * L["patch_rw"] <= 128 and (L["rh2"], L["rw2"]) == (L["patch_rh"], L["patch_rw"])
    assert pl["bytes_linked"] <= 14.8e9          # 15.9e9 before these links (fp32 image input)
    # explicit requests reach the chains the model declines: a basic block of ResNet-18, a fire module
    r = graphs.resnet18()
    g2, _ = compiled(r, 2, links=[["s1b1.c1", "s1b1.c2", "s1b1.add"]])
    L = [l for l in g2.plan()["launches"] if l["kind"] == "gemm2"]
    assert len(L) == 1 and (L[0]["k"], L[0]["k2"]) == (3, 3) and (L[0]["rh2"], L[0]["rw2"]) == (L[0]["patch_rh"] - 2, L[0]["patch_rw"] - 2)
    q = graphs.squeezenet11()
    g3, _ = compiled(q, 2, links=[["f3.sq", "f3.e1", "f3.e3", "f3.cat"]])
    L = [l for l in g3.plan()["launches"] if l["kind"] == "gemm2"]
    assert len(L) == 1 and L[0]["cmid"] == 32 and L[0]["n1pad"] == 64 and L[0]["K"] == 256


# ---- graph image (Section 6: the optimised model as a stored executable) ---------------------------------------
def _fnv1a(b: bytes) -> int:
    h = 1469598103934665603
    for x in b:
        h = ((h ^ x) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    return h


@pytest.mark.parametrize("name,batch", [("single_chain", 1), ("mobilenet_v1", 4), ("resnet18", 2), ("squeezenet11", 2)])
def test_graph_image_round_trip_gives_the_same_plan(name, batch):
    spec = getattr(graphs, name)()
    g, _ = compiled(spec, batch)
    img = g.save()
    g2, ws = xb.Graph.load(img)
    assert g2.plan_text() == g.plan_text()          # same chains, tiles, offsets and packed parameters' layout
    assert ws == g.plan()["workspace_bytes"]
    assert g2.save() == img                         # the image of the loaded graph is the same bytes


def test_graph_image_keeps_requests_and_build_state():
    spec = graphs.mobilenet_v1(hw=64, width=0.5, classes=16)
    P = graphs.make_params(spec)
    g, ids = graph_from_spec(spec, P)
    g.link([ids["dw3"], ids["pw3"]])
    g.split(ids["pw3.relu6"], parts_outc=2)
    g2, ws = xb.Graph.load(g.save())                # saved before compile: comes back in build state
    assert ws == 0
    with pytest.raises(xb.XenosError) as e:
        g2.plan()
    assert e.value.code == xb.E_STATE
    g.compile(2, xb.PRECISION_BF16_TENSOR)
    g2.compile(2, xb.PRECISION_BF16_TENSOR)
    assert g2.plan_text() == g.plan_text()
    L = [l for l in g2.plan()["launches"] if l.get("a0") == "dw"]
    assert len(L) == 1 and L[0]["n_tiles"] == 2     # the one explicit link, with its explicit split


def test_graph_image_rejects_what_is_not_an_intact_image():
    g, _ = compiled(graphs.single_chain(), 1)
    img = g.save()
    def bad(b):
        with pytest.raises(xb.XenosError) as e:
            xb.Graph.load(b)
        assert e.value.code == xb.E_INVALID
    bad(b"")
    bad(img[:16])
    bad(b"NOTANIMG" + img[8:])
    for cut in (1, 8, 9, len(img) // 2):
        bad(img[:-cut])                             # truncated
    flipped = bytearray(img); flipped[len(img) // 3] ^= 0x40
    bad(bytes(flipped))                             # altered: checksum
    def resum(b):
        return bytes(b[:-8]) + _fnv1a(bytes(b[:-8])).to_bytes(8, "little")
    v2 = bytearray(img); v2[8] = 2
    bad(resum(v2))                                  # another version, intact checksum
    # an intact checksum over fields that do not fit: a tensor count larger than the image
    huge = bytearray(img); huge[32:40] = (1 << 40).to_bytes(8, "little")
    bad(resum(huge))
    # ... and an operator that names a tensor that does not exist (first tensor's producer field)
    idx = bytearray(img)
    off = 8 + 4 + 20 + 8 + 16                       # magic, version, hw, tensor count, c h w is_vec of tensor 0
    idx[off:off + 4] = (12345).to_bytes(4, "little")
    bad(resum(idx))
    assert xb.Graph.load(img)[0].plan_text() == g.plan_text()     # the untouched image still loads


def test_image_convolution_and_max_pool_link_by_measured_cost():
    """At batch 8 and above an image convolution and its max pool run as two kernels (measured faster), unless the image is
    wider than 256 pixels or the link is requested; at small batch they are linked.  An unlinked image convolution's tiles
    keep their input patch within the copy engine's 256 x 256 box, also for a 512 x 512 image."""
    spec = graphs.resnet18()
    def first_chain(batch, **kw):
        pl = compiled(spec, batch, **kw)[0].plan()
        return [pl["nodes"][i]["kind"] for i in pl["chains"][0]["nodes"]]
    assert first_chain(1) == ["conv", "maxpool"]
    assert first_chain(32) == ["conv"]
    assert first_chain(32, links=[["stem", "mp"]]) == ["conv", "maxpool"]
    pl = compiled(graphs.resnet50_stress(), 8)[0].plan()
    assert [pl["nodes"][i]["kind"] for i in pl["chains"][0]["nodes"]] == ["conv", "maxpool"]
    pl = compiled(graphs.resnet50_stress(), 8, linked=False)[0].plan()
    stem = pl["launches"][0]
    assert stem["a0"] == "stem" and (stem["patch_rw"] - 1) * 2 + 18 <= 256 and stem["hstages"] >= 2      # hstages: patches by TMA
