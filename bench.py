"""Benchmark: images/s of one linked CNN graph on B200, with roofline and CPU-oracle context.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

A step is one pass of the whole hot path (every linked chain of the graph) over one batch of
seeded synthetic images.  Default workload: MobileNetV1-style depthwise-separable graph,
width 1.0, 224x224, batch 32, bf16 activations with fp32 accumulation, linked execution.
Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from xenos_workloads import graphs  # noqa: E402
from xenos_workloads.feed import graph_from_spec  # noqa: E402

WORKLOADS = {
    "mobilenet_v1_b32": (1, 32), "mobilenet_v1_b1": (1, 1),
    "resnet18_b32": (2, 32), "resnet18_b1": (2, 1),
    "squeezenet11_b32": (3, 32), "squeezenet11_b1": (3, 1),
    "resnet50_stress_b64": (4, 64), "single_chain_b1": (0, 1),
    "resnet50_stress_b8": (4, 8),       # the stress graph at a batch small enough for a profiler capture
    # the paper's operator micro-benchmarks (Table 4): the first two exercise linking (other arm: unlinked), the
    # last two the split (other arm: the coarsest split the kernels allow, 256-wide channel tiles, K uncut)
    "op_cbr_maxpool_b32": ("cbr_maxpool", 32), "op_cbr_avgpool_b32": ("cbr_avgpool", 32),
    "op_fc_b32": ("fc", 32), "op_cbr_b32": ("cbr", 32),
    "op_cbr_maxpool_b1": ("cbr_maxpool", 1), "op_cbr_avgpool_b1": ("cbr_avgpool", 1),
    "op_fc_b1": ("fc", 1), "op_cbr_b1": ("cbr", 1),
}
SPLIT_WORKLOADS = {"fc": "fc", "cbr": "c"}      # operator benchmark -> the operator whose split the other arm coarsens


def workload_spec(key):
    return graphs.operator_benchmark(key) if isinstance(key, str) else graphs.config(key)[0]
L2_FLUSH_BYTES = 256 << 20
MIN_TIMED_SECONDS = 0.3      # the K timed steps are repeated until the timed region covers at least this long


def ncu_traffic_table():
    """Measured DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, averaged over the launches of
    one step) by (workload, arm, kernel), from the table kept beside the ncu summaries.  A row is removed there
    whenever its kernel changes after the capture, and the bench then reports null."""
    table = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic_table.txt")
    if os.path.exists(path):
        for line in open(path):
            f = line.split()
            if len(f) >= 4 and not line.startswith("#"):
                table[(f[0], f[1], f[2])] = float(f[3])
    return table


def max_over_ranks(value: float, device: str) -> float:
    """The slowest rank decides: replicas run independently, the job is as fast as its last replica."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(world: int, batch: int, steps: int, total_ms: float) -> float:
    """Images per second of all replicas together: every rank processes `batch` images per step."""
    return world * batch * steps / (total_ms * 1e-3)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = "clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
            "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.t.join(timeout=2)
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                mhz.append(float(r[0])); mx = float(r[1])
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=float(np.median(mhz)) if mhz else None, sm_max_mhz=mx, reasons=sorted(reasons), samples=len(mhz))


def reference_arm(args, spec, batch):
    """Times the CPU oracle (as it stands) on the host cores: one step = a bounded sample of the batch."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as xo
    from oracle import interp
    P = graphs.make_params(spec)
    sample = min(batch, args.ref_images)
    x = graphs.make_input(spec, sample)
    for _ in range(min(args.warmup, 1)):
        interp.run_graph(spec, P, x[:1])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        interp.run_graph(spec, P, x)
    dt = time.perf_counter() - t0
    val = sample * args.steps / dt
    line = dict(impl="reference", metric="images/sec per linked CNN graph", value=val, unit="images/s", n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * dt / args.steps, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f32", data="synthetic",
                config=dict(workload=args.workload, graph=spec.name, global_batch=batch, mode="cpu oracle, one operator at a time"),
                cpu_baseline=dict(value=val, unit="images/s", cores=xo.num_threads(), kind="oracle",
                                  sample=f"{sample} of {batch} images per step"),
                e2e=dict(value=val, unit="images/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="xenos")
    ap.add_argument("--workload", default="mobilenet_v1_b32", choices=sorted(WORKLOADS))
    ap.add_argument("--ref-images", type=int, default=8, help="images per step of the CPU oracle arm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="repeat the K timed steps until they cover this long (0: one pass, for profiler captures)")
    ap.add_argument("--unlinked", action="store_true", help="time the unlinked execution as the main arm")
    args = ap.parse_args()
    cfg, batch = WORKLOADS[args.workload]
    spec = workload_spec(cfg)
    if args.impl == "reference":
        reference_arm(args, spec, batch)
        return

    import torch
    import torch.distributed as dist
    from paper_2302_00282_b200 import binding as xb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    fp32 = spec.precision == "fp32"
    P = graphs.make_params(spec)
    x = graphs.make_input(spec, batch)

    # images enter as NCHW; feature maps with 8 or more channels enter as NHWC bf16, the layout between kernels
    nhwc = (not fp32) and spec.in_shape[0] >= 8
    split_op = SPLIT_WORKLOADS.get(cfg) if isinstance(cfg, str) else None
    other_name = "coarsest split" if split_op else "unlinked"

    def make(linked):
        g, ids = graph_from_spec(spec, P, in_dtype=xb.DTYPE_F32 if fp32 else xb.DTYPE_BF16,
                                 in_layout=xb.LAYOUT_NHWC if nhwc else xb.LAYOUT_NCHW)
        if split_op:
            # main arm: the automatic split; other arm: as few, as wide tiles as the kernels allow
            g.link()
            if not linked:
                cout = [o for o in spec.ops if o["name"] == split_op][0]["cout"]
                g.split(ids[split_op], parts_outc=-(-cout // 256), parts_k=1)
        elif linked:
            g.link()
        nbytes = g.compile(batch, xb.PRECISION_FP32_CUDA_CORE if fp32 else xb.PRECISION_BF16_TENSOR)
        ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        g.bind(ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
        return g, ws

    stream = torch.cuda.current_stream().cuda_stream
    x_nchw = x
    if nhwc:
        x = np.ascontiguousarray(x.transpose(0, 2, 3, 1))
    x_host = torch.from_numpy(x) if fp32 else torch.from_numpy(x).to(torch.bfloat16)
    x_pin = x_host.pin_memory()
    x_dev = x_host.cuda()
    oshape = spec.shapes[spec.output]
    if len(oshape) == 1:
        out_dev = torch.empty((batch, oshape[0]), dtype=torch.float32, device="cuda")
    elif fp32:
        out_dev = torch.empty((batch,) + tuple(oshape), dtype=torch.float32, device="cuda")
    else:
        out_dev = torch.empty((batch, oshape[1], oshape[2], oshape[0]), dtype=torch.bfloat16, device="cuda")
    out_pin = torch.empty_like(out_dev, device="cpu").pin_memory()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def time_steps(g, steps, warmup, e2e=False):
        for _ in range(warmup):
            g.run(batch, [x_dev.data_ptr()], [out_dev.data_ptr()], stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        for i in range(steps):
            flush.fill_(i & 0xFF)                    # evict L2 between timed steps (outside the timed interval)
            starts[i].record()
            if e2e:
                x_dev.copy_(x_pin, non_blocking=True)
            g.run(batch, [x_dev.data_ptr()], [out_dev.data_ptr()], stream)
            if e2e:
                out_pin.copy_(out_dev, non_blocking=True)
            ends[i].record()
        torch.cuda.synchronize()
        g.status(stream)
        total_ms = sum(s.elapsed_time(e) for s, e in zip(starts, ends))
        if world > 1:
            total_ms = max_over_ranks(total_ms, "cuda")
            dist.barrier()
        torch.cuda.synchronize()
        return total_ms

    def time_e2e(g, steps, warmup):
        """The serving loop a user of the library writes: step i's input goes host -> device (pinned memory, a
        copy stream, two device buffers) while step i-1 computes; every step's result is read back.  One event
        pair brackets the whole loop; the L2 flush between steps runs inside it."""
        for _ in range(warmup):
            g.run(batch, [x_dev.data_ptr()], [out_dev.data_ptr()], stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        copy_stream = torch.cuda.Stream()
        bufs = [x_dev, torch.empty_like(x_dev)]
        ready = [torch.cuda.Event() for _ in range(2)]
        free = [torch.cuda.Event() for _ in range(2)]
        main = torch.cuda.current_stream()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for b in range(2):
            free[b].record(main)
        t0.record(main)
        copy_stream.wait_event(t0)
        for i in range(steps):
            b = i & 1
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(free[b])           # the step that last read this buffer is done
                bufs[b].copy_(x_pin, non_blocking=True)
                ready[b].record(copy_stream)
            main.wait_event(ready[b])
            flush.fill_(i & 0xFF)
            g.run(batch, [bufs[b].data_ptr()], [out_dev.data_ptr()], stream)
            free[b].record(main)
            out_pin.copy_(out_dev, non_blocking=True)
        t1.record(main)
        torch.cuda.synchronize()
        g.status(stream)
        total_ms = t0.elapsed_time(t1)
        if world > 1:
            total_ms = max_over_ranks(total_ms, "cuda")
            dist.barrier()
        torch.cuda.synchronize()
        return total_ms

    g_main, ws_main = make(not args.unlinked)
    sampler = ClockSampler(local)
    sampler.start()
    # K timed steps per repeat; repeats until the timed region is long enough for the clock sampler and for a
    # stable mean.  ms_per_step is the mean over all repeats, the median of the repeats is reported beside it.
    rep_ms = [time_steps(g_main, args.steps, args.warmup)]
    repeats = int(min(200, max(1, np.ceil(args.min_seconds * 1e3 / max(rep_ms[0], 1e-3)))))
    for _ in range(repeats - 1):
        rep_ms.append(time_steps(g_main, args.steps, 0))
    clocks = sampler.stop()
    total_ms = float(np.mean(rep_ms))
    value = whole_job_throughput(world, batch, args.steps, total_ms)
    e2e_steps = max(8, args.steps // 2)
    e2e_ms = time_e2e(g_main, e2e_steps, 3)
    e2e_val = world * batch * e2e_steps / (e2e_ms * 1e-3)

    # the other arm (unlinked when the main arm is linked) on the same inputs, fewer steps
    g_other, ws_other = make(args.unlinked)
    osteps = max(3, args.steps // 4)
    other_ms = time_steps(g_other, osteps, 3)
    other_val = world * batch * osteps / (other_ms * 1e-3)

    # per-launch device times of the main arm -> roofline of the dominant kernel
    plan = g_main.plan()
    reps = 5
    acc = np.zeros(len(plan["launches"]))
    for i in range(reps + 1):
        flush.fill_(i)
        ms = g_main.profile(batch, [x_dev.data_ptr()], [out_dev.data_ptr()], stream)
        if i:
            acc += np.array(ms)
    acc /= reps
    peaks = measured_peaks()
    by_kind = {}
    for L, ms in zip(plan["launches"], acc):
        d = by_kind.setdefault(L["kind"], dict(ms=0.0, bytes=0.0, flops=0.0, launches=0))
        d["ms"] += float(ms); d["bytes"] += L["bytes"]; d["flops"] += L["flops"]; d["launches"] += 1
    dom = max(by_kind, key=lambda k: by_kind[k]["ms"])
    dk = by_kind[dom]
    t_mem = dk["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_tc = dk["flops"] / (peaks["bf16_tflops"] * 1e12)
    # In-stream duration of the dominant kernel's launches: the timed step minus the other kernels' share of it
    # (shares from the serialised per-launch times; when the step runs one kernel only, as the linked tensor-core
    # graphs do, this is the timed step itself).
    all_ms = sum(d["ms"] for d in by_kind.values())
    step_ms = total_ms / args.steps
    dom_ms_in_stream = step_ms * dk["ms"] / all_ms
    if t_tc > t_mem and not fp32:
        roof = dict(bound="tensor", achieved=dk["flops"] / (dom_ms_in_stream * 1e-3) / 1e12, peak=peaks["bf16_tflops"], unit="TFLOP/s")
        serial = dk["flops"] / (dk["ms"] * 1e-3) / 1e12
    else:
        roof = dict(bound="hbm", achieved=dk["bytes"] / (dom_ms_in_stream * 1e-3) / 1e9, peak=peaks["hbm_gbs"], unit="GB/s")
        serial = dk["bytes"] / (dk["ms"] * 1e-3) / 1e9
    traffic = ncu_traffic_table().get((args.workload, "unlinked" if args.unlinked else "linked", dom))
    roof.update(frac=roof["achieved"] / roof["peak"], traffic=traffic, kernel=dom, launches_per_step=dk["launches"],
                avg_launch_us=1e3 * dom_ms_in_stream / dk["launches"], peak_source=peaks["source"],
                algorithmic_bytes_per_launch=dk["bytes"] / dk["launches"],
                algorithmic_bytes_per_step=dk["bytes"], flops_per_step=dk["flops"],
                timing="launches in the stream of the timed step (CUDA events around each step)",
                serialised=dict(achieved=serial, frac=serial / roof["peak"], avg_launch_us=1e3 * dk["ms"] / dk["launches"],
                                note="each launch timed alone between its own events: no overlap of one launch's "
                                     "set-up with its predecessor's drain; the per-chain list uses these times as shares"))
    chains = []
    for c in plan["chains"]:
        ms = float(sum(acc[i] for i in c["launches"]))
        tm, tt = c["bytes_linked"] / (peaks["hbm_gbs"] * 1e9), c["flops"] / (peaks["bf16_tflops"] * 1e12)
        # in-stream time of the chain = its share of the serialised times, applied to the timed step
        us = 1e3 * step_ms * ms / all_ms if all_ms > 0 else 0.0
        chains.append(dict(id=c["id"], kind=c["kind"], us=us, us_serialised=1e3 * ms, share=ms / all_ms if all_ms > 0 else None,
                           bound="tensor" if tt > tm else "hbm", roofline_us=max(tm, tt) * 1e6,
                           frac=(max(tm, tt) * 1e6) / us if us > 0 else None))

    line = dict(metric="images/sec per linked CNN graph", value=value, unit="images/s", n_gpus=world, steps=args.steps,
                warmup=args.warmup, ms_per_step=total_ms / args.steps, ms_per_step_median=float(np.median(rep_ms)) / args.steps,
                repeats=repeats, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f32" if fp32 else "bf16", data="synthetic",
                config=dict(workload=args.workload, graph=spec.name, global_batch=batch * world, input=list(spec.in_shape),
                            mode="unlinked" if args.unlinked else "linked", l2="flushed between timed steps (256 MiB write)",
                            parallelism="replicas only" if world > 1 else "single GPU"),
                clocks=clocks,
                e2e=dict(value=e2e_val, unit="images/s", h2d_bytes_per_step=x_pin.numel() * x_pin.element_size(),
                         d2h_bytes_per_step=out_pin.numel() * out_pin.element_size(), steps=e2e_steps,
                         loop="copy of step i+1 overlaps compute of step i (two device buffers); L2 flush inside the timed loop"),
                gpu_launches=g_main.launch_count() * args.steps * repeats,
                roofline=roof,
                linked_vs_unlinked=dict(other_mode="linked" if args.unlinked else other_name, other_value=other_val,
                                        speedup=(value / other_val) if not args.unlinked else (other_val / value),
                                        launches_linked=(g_other if args.unlinked else g_main).launch_count(),
                                        launches_unlinked=(g_main if args.unlinked else g_other).launch_count(),
                                        model_bytes_linked=plan["bytes_linked"], model_bytes_unlinked=plan["bytes_unlinked"]),
                chains=chains)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle as xo
        from oracle import interp
        # a bounded sample of the same workload: whole passes of up to 16 images until about 10 s of CPU work
        sample = min(batch, 16)
        interp.run_graph(spec, P, x_nchw[:1])
        passes, t0 = 0, time.perf_counter()
        while True:
            interp.run_graph(spec, P, x_nchw[:sample])
            passes += 1
            dt = time.perf_counter() - t0
            if dt >= 10.0 or passes >= 64:
                break
        line["cpu_baseline"] = dict(value=sample * passes / dt, unit="images/s", cores=xo.num_threads(), kind="oracle",
                                    sample=f"{sample} of {batch} images x {passes} passes, {dt:.1f} s")
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
