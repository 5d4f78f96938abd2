"""The entry point for callers that cannot allocate device memory.

Some users of this library run where the device allocator is off limits: a plugin inside an
application that owns all device memory, or a real-time loop that must not call cudaMalloc.
For them xenos_graph_run_builtin_scratch runs a compiled graph with a fixed 16 MiB workspace that
is part of the library itself.  These tests check, through the C ABI, that its results equal those
of the ordinary bind + run path on two calls in a row (the shared array keeps the previous call's
contents, so the second call is the one that would expose stale state), that two graphs can take
turns on the array, and that a graph too large for it is refused with a clear message.
"""
import numpy as np
import pytest

from oracle import interp
from xenos_workloads import graphs
from xenos_workloads.feed import graph_from_spec

from paper_2302_00282_b200 import binding as xb


def test_oversized_graph_is_refused_with_both_sizes():
    spec = graphs.mobilenet_v1()                 # batch 32 needs far more than 16 MiB
    P = graphs.make_params(spec)
    g, _ = graph_from_spec(spec, P)
    g.link()
    need = g.compile(32, xb.PRECISION_BF16_TENSOR)
    assert need > (16 << 20)
    with pytest.raises(xb.XenosError) as e:
        g.run_builtin_scratch(32, [256], [256])
    assert e.value.code == xb.E_WORKSPACE
    assert str(need) in str(e.value) and str(16 << 20) in str(e.value)


@pytest.mark.gpu
def test_builtin_scratch_on_an_unbound_graph_and_with_a_partial_batch():
    """compile only, no bind: the entry point needs no caller workspace at all; and batch < max_batch."""
    import torch
    from gpu_util import GpuGraph, abs_err_scaled

    spec = graphs.mobilenet_v1(hw=32, width=0.25, classes=16)
    P = graphs.make_params(spec)
    x = graphs.make_input(spec, 3)
    g, _ = graph_from_spec(spec, P)
    g.link()
    assert g.compile(8, xb.PRECISION_BF16_TENSOR) <= (16 << 20)
    stream = torch.cuda.current_stream().cuda_stream
    xin = torch.from_numpy(x).cuda()
    out = torch.full((3, 16), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):
        g.run_builtin_scratch(3, [xin.data_ptr()], [out.data_ptr()], stream)
        y = out.cpu().numpy()
        assert not np.isnan(y).any()
        assert abs_err_scaled(y, interp.run_graph(spec, P, x)) <= 2e-2
    ref = GpuGraph(spec, P, 8, linked=True).run(x)
    assert np.array_equal(y, ref)
    with pytest.raises(xb.XenosError) as e:
        g.run(3, [xin.data_ptr()], [out.data_ptr()], stream)      # still unbound for the ordinary path
    assert e.value.code == xb.E_STATE


@pytest.mark.gpu
def test_builtin_scratch_matches_bound_workspace_twice_in_a_row():
    import torch
    from gpu_util import GpuGraph, abs_err_scaled, rel_err_fp32

    stream = torch.cuda.current_stream().cuda_stream
    cases = [(graphs.single_chain(), 2, True), (graphs.mobilenet_v1(hw=64, width=0.5, classes=16), 3, True),
             (graphs.squeezenet11(hw=63, classes=24, scale=2), 2, False)]
    built = []
    for spec, batch, linked in cases:
        P = graphs.make_params(spec)
        x = graphs.make_input(spec, batch)
        gg = GpuGraph(spec, P, batch, linked=linked)          # ordinary path: caller-owned workspace
        ref = gg.run(x)
        o = interp.run_graph(spec, P, x)
        built.append((spec, gg, x, ref, o))

    def run_builtin(gg, x):
        xin = gg.upload(x)
        out = gg.alloc_out(x.shape[0])
        gg.g.run_builtin_scratch(x.shape[0], [xin.data_ptr()], [out.data_ptr()], stream)
        y = out.float().cpu().numpy()
        if not gg.vec and not gg.fp32:
            y = np.ascontiguousarray(y.transpose(0, 3, 1, 2))
        return y

    # two calls in a row per graph, then the graphs take turns (each turn re-uploads parameters)
    for rnd in range(2):
        for spec, gg, x, ref, o in built:
            for call in range(2):
                y = run_builtin(gg, x)
                assert not np.isnan(y).any()
                if gg.fp32:
                    assert rel_err_fp32(y, ref) <= 1e-4 and rel_err_fp32(y, o) <= 1e-4
                else:
                    assert abs_err_scaled(y, ref) <= 2e-2 and abs_err_scaled(y, o) <= 2e-2
                assert np.array_equal(y, ref), (spec.name, rnd, call)   # same kernels, same plan: same bits
    # the ordinary binding was left untouched
    spec, gg, x, ref, o = built[1]
    assert np.array_equal(gg.run(x), ref)
