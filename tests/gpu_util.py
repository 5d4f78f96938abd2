"""Helpers for the GPU parity tests: run a workload graph through the C ABI on cuda:0 and
return the result as an NCHW fp32 numpy array comparable with the CPU oracle's."""
from __future__ import annotations

import json
import os

import numpy as np

def log(rec: dict):
    """Appends one record to the file named by XENOS_PARITY_LOG (no log when the variable is unset)."""
    path = os.environ.get("XENOS_PARITY_LOG")
    if not path:
        return
    try:
        os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
        with open(path, "a") as f:
            f.write(json.dumps(rec) + "\n")
    except OSError:
        pass


def to_nhwc_bf16(x_nchw: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x_nchw.transpose(0, 2, 3, 1))).to(torch.bfloat16)


class GpuGraph:
    """Compiled + bound graph with its device buffers (all memory owned by PyTorch)."""

    def __init__(self, spec, params, max_batch, linked=True, in_mode="f32_nchw", splits=(), links=None):
        import torch
        from paper_2302_00282_b200 import binding as xb
        from xenos_workloads.feed import graph_from_spec
        self.xb, self.torch, self.spec = xb, torch, spec
        dt, lay = {"f32_nchw": (xb.DTYPE_F32, xb.LAYOUT_NCHW), "bf16_nchw": (xb.DTYPE_BF16, xb.LAYOUT_NCHW),
                   "bf16_nhwc": (xb.DTYPE_BF16, xb.LAYOUT_NHWC)}[in_mode]
        self.in_mode = in_mode
        self.g, self.ids = graph_from_spec(spec, params, in_dtype=dt, in_layout=lay)
        if links is not None:
            for chain in links:
                self.g.link([self.ids[n] for n in chain])
        elif linked:
            self.g.link()
        for name, kw in splits:
            self.g.split(self.ids[name], **kw)
        self.fp32 = spec.precision == "fp32"
        nbytes = self.g.compile(max_batch, xb.PRECISION_FP32_CUDA_CORE if self.fp32 else xb.PRECISION_BF16_TENSOR)
        self.max_batch = max_batch
        self.ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        # poison the workspace so that an unwritten intermediate shows up as NaN
        self.ws.fill_(0xFF)
        self.stream = torch.cuda.current_stream().cuda_stream
        self.g.bind(self.ws.data_ptr(), self.ws.numel(), self.stream)
        oshape = spec.shapes[spec.output]
        self.vec = len(oshape) == 1
        self.oshape = oshape

    def upload(self, x_nchw: np.ndarray):
        torch = self.torch
        if self.in_mode == "f32_nchw":
            return torch.from_numpy(np.ascontiguousarray(x_nchw, np.float32)).cuda()
        if self.in_mode == "bf16_nchw":
            return torch.from_numpy(np.ascontiguousarray(x_nchw, np.float32)).to(torch.bfloat16).cuda()
        return to_nhwc_bf16(x_nchw).cuda()

    def alloc_out(self, batch):
        torch = self.torch
        if self.vec:
            return torch.full((batch, self.oshape[0]), float("nan"), dtype=torch.float32, device="cuda")
        c, h, w = self.oshape
        if self.fp32:
            return torch.full((batch, c, h, w), float("nan"), dtype=torch.float32, device="cuda")
        return torch.full((batch, h, w, c), float("nan"), dtype=torch.bfloat16, device="cuda")

    def run(self, x_nchw: np.ndarray) -> np.ndarray:
        torch = self.torch
        batch = x_nchw.shape[0]
        xin = self.upload(x_nchw)
        out = self.alloc_out(batch)
        self.g.run(batch, [xin.data_ptr()], [out.data_ptr()], self.stream)
        self.g.status(self.stream)
        y = out.float().cpu().numpy()
        if not self.vec and not self.fp32:
            y = np.ascontiguousarray(y.transpose(0, 3, 1, 2))
        return y


def rel_err_fp32(g: np.ndarray, o: np.ndarray) -> float:
    """max_i |g_i - o_i| / max(|o_i|, 1e-2 * max|o|): elementwise relative error, with the
    denominator floored where the oracle's own fp32 rounding already exceeds 1e-4 relative."""
    floor = 1e-2 * float(np.abs(o).max())
    return float((np.abs(g - o) / np.maximum(np.abs(o), max(floor, 1e-30))).max())


def abs_err_scaled(g: np.ndarray, o: np.ndarray) -> float:
    """max_i |g_i - o_i| / max_i |o_i| (the bf16 tensor-core bound is 2e-2)."""
    return float(np.abs(g - o).max() / max(float(np.abs(o).max()), 1e-30))
