#!/usr/bin/env python
"""Benchmark of fused operator chains on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one run of a whole fused chain (every kernel of its plan) on one batch of seeded
synthetic input.  The headline workload is the memory-bound chain (affine, GELU, row softmax,
row layer normalisation on an fp32 [8192,4096] tensor); throughput is algorithmic bytes per
second (inputs read once, outputs written once).  Contraction chains report TFLOP/s.
With N > 1 every rank runs an independent replica on its own GPU (the chains do not shard
across devices); the value is the sum over ranks divided by the slowest rank's time.
Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from workloads import configs  # noqa: E402

WORKLOADS = {
    "c2_softmax_layernorm_chain": dict(bound="hbm", sample=dict(r=8192)),
    "c3_gemm_bf16_gelu_residual": dict(bound="tensor", sample=dict(m=2048)),
    "c4_conv_bn_relu_bf16": dict(bound="tensor", sample=dict(n=8)),
    "c1_gemm_bias_relu_f32": dict(bound="tensor", sample=dict()),
    # operator classes beyond the five configurations: a layout transform and the case-study chain with dropout
    "transpose_bias_relu": dict(bound="hbm", sample=dict(r=4096)),
    "matmul_dropout_mean_softmax": dict(bound="tensor", sample=dict(m=1024)),
    "conv_block": dict(bound="tensor", sample=dict(n=4)),
    "dwconv_bn_relu": dict(bound="hbm", sample=dict(n=8)),
    "topk_bias_relu": dict(bound="hbm", sample=dict(r=2048)),
    "mbconv_block": dict(bound="hbm", sample=dict(n=4)),
}
HEADLINE = "c2_softmax_layernorm_chain"


def kernel_fingerprint(g):
    """Hash of the generated source of every kernel of a graph: changes whenever a kernel changes."""
    import hashlib
    h = hashlib.sha256()
    for i in range(g.num_kernels):
        h.update(g.kernel_source(i).encode())
    return h.hexdigest()[:16]


def recorded_traffic(name, fingerprint):
    """DRAM bytes per launch from the committed ncu summary, or None once the kernels have changed since."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    rec = json.load(open(path)).get(name)
    if not rec or rec.get("fingerprint") != fingerprint:
        return None
    return rec["dram_bytes_per_step"]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm": p["hbm_gbs"], "tensor": p["bf16_tflops"], "tensor_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm": 6650.0, "tensor": 1590.0, "tensor_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        q = "clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
            "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = max(mx, float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx or None, "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_value(bound, bytes_per_rank, flops_per_rank, world, slowest_seconds_per_step):
    """Replicas: every rank processes the same units; the job's rate is all units over the slowest rank's time."""
    return metric_of(bound, bytes_per_rank * world, flops_per_rank * world, slowest_seconds_per_step)


def metric_of(bound, bytes_, flops, seconds):
    if bound == "hbm":
        return bytes_ / seconds / 1e9, "GB/s"
    return flops / seconds / 1e12, "TFLOP/s"


def oracle_arm(name, steps, warmup):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload."""
    import oracle
    from workloads import tensors
    info = WORKLOADS[name]
    spec, laws = configs.get_config(name, **info["sample"])
    t = configs.draw_inputs(spec, laws, 0)
    ins = {n: tensors.as_float64(t[n], d) for n, d, _ in configs.parse_inputs(spec)}
    g = oracle.parse(spec)
    in_bytes = sum(t[n].nbytes for n in t)
    out_elems = sum(int(np.prod(g.nodes[o].shape)) for o, _ in g.outputs)
    out_bytes = sum(int(np.prod(g.nodes[o].shape)) * (2 if d == "bf16" else 4) for o, d in g.outputs)
    flops = 0.0
    for node in g.nodes.values():
        if node.op == "gemm":
            flops += 2.0 * g.nodes[node.args[0]].shape[0] * g.nodes[node.args[0]].shape[1] * node.shape[1]
        elif node.op == "conv2d":
            w = g.nodes[node.args[1]].shape
            flops += 2.0 * np.prod(node.shape) * w[1] * w[2] * w[3]
    for _ in range(warmup):
        oracle.run(g, ins)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.run(g, ins)
    dt = (time.perf_counter() - t0) / steps
    value, unit = metric_of(info["bound"], in_bytes + out_bytes, flops, dt)
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    sample = ", ".join(f"{k}={v}" for k, v in info["sample"].items()) or "full size"
    return dict(value=value, unit=unit, cores=cores, kind="oracle", sample=f"{name} at {sample} ({out_elems} output elements per step)",
                ms_per_step=dt * 1e3)


def run_gpu(name, steps, warmup, rank, world, device, tune=0):
    import torch
    import paper_2506_10401_b200 as hct
    from tests import parity

    info = WORKLOADS[name]
    spec, laws = configs.get_config(name)
    host = configs.draw_inputs(spec, laws, 0)
    ins = parity.to_device(spec, host, f"cuda:{device}")
    # with --tune N the schedule is picked by measurement (set-up, untimed); the default is the fixed rules
    g = hct.FusedGraph.autotuned(spec, ins, device, max_trials=tune) if tune > 0 else hct.FusedGraph(spec, device)
    outs = g.alloc_outputs()
    bytes_, flops = g.cost()
    stream = torch.cuda.current_stream(device)
    flush = torch.empty(192 * 1024 * 1024, dtype=torch.uint8, device=f"cuda:{device}")  # larger than the 126 MB L2

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(device)

    for _ in range(max(warmup, 3)):
        flush.zero_()
        g.run(ins, outs, stream)
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    with ClockSampler(device) as clocks:
        for a, b in ev:
            flush.zero_()           # evict the previous step's data from L2; not timed
            a.record(stream)
            g.run(ins, outs, stream)
            b.record(stream)
        barrier()
    g.status()
    per_step = [a.elapsed_time(b) * 1e-3 for a, b in ev]
    dev_s = float(np.sum(per_step))

    # end to end: pinned host inputs -> device, run, result back to the host, every step.  The three
    # phases of consecutive steps overlap (copy-in, compute and copy-out streams, two sets of device
    # buffers): PCIe is full duplex, so step i+1's inputs travel while step i's result returns.
    specs_in = configs.parse_inputs(spec)
    pinned = [torch.from_numpy(host[n].view(np.int16) if d == "bf16" else host[n]).pin_memory() for n, d, _ in specs_in]
    dev_in = [[torch.empty_like(t, device=f"cuda:{device}") for t in pinned] for _ in range(2)]
    run_in = [[t.view(torch.bfloat16) if d == "bf16" else t for t, (_, d, _) in zip(buf, specs_in)] for buf in dev_in]
    dev_out = [outs, g.alloc_outputs()]
    host_out = [[torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs] for _ in range(2)]
    h2d = sum(t.numel() * t.element_size() for t in pinned)
    d2h = sum(t.numel() * t.element_size() for t in host_out[0])
    e2e_steps = max(4, min(steps, 8))
    s_in, s_run, s_out = (torch.cuda.Stream(device) for _ in range(3))
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_run = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_loop(n):
        for i in range(n):
            b = i % 2
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_run[b])      # the kernels of step i-2 have read this input set
                for src, dst in zip(pinned, dev_in[b]):
                    dst.copy_(src, non_blocking=True)
                ev_in[b].record(s_in)
            s_run.wait_event(ev_in[b])
            if i >= 2:
                s_run.wait_event(ev_out[b])         # step i-2's result has left this output set
            g.run(run_in[b], dev_out[b], s_run)
            ev_run[b].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[b])
                for src, dst in zip(dev_out[b], host_out[b]):
                    dst.copy_(src, non_blocking=True)
                ev_out[b].record(s_out)

    e2e_loop(2)
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(s_in)
    e2e_loop(e2e_steps)
    s_out.wait_stream(s_in)
    s_out.wait_stream(s_run)
    b.record(s_out)
    barrier()
    e2e_s = a.elapsed_time(b) * 1e-3 / e2e_steps
    g.status()

    dev_s, e2e_s = max_over_ranks([dev_s, e2e_s], f"cuda:{device}")
    value, unit = whole_job_value(info["bound"], bytes_, flops, world, dev_s / steps)
    e2e_v, _ = whole_job_value(info["bound"], bytes_, flops, world, e2e_s)
    kern_s = float(np.mean(per_step))
    return dict(value=value, unit=unit, ms_per_step=dev_s / steps * 1e3, bytes=bytes_, flops=flops, kernel_s=kern_s,
                fingerprint=kernel_fingerprint(g),
                kernels=g.num_kernels, clocks=clocks.summary(), e2e=dict(value=e2e_v, unit=unit, h2d_bytes_per_step=h2d,
                                                                         d2h_bytes_per_step=d2h), plan=g.plan,
                schedule=g.schedule)


def run_sweep(steps, warmup, device, out_path=None, tune=0):
    """The 200 random operator DAGs: per-graph time against its own roofline, and class aggregates.

    Inputs are drawn on the device from the same laws (normal / uniform with the recipe's mean and
    spread, seeded per graph) because host-side generation of ~10^10 elements would dominate the run;
    parity on these graphs is covered by the tests with the counter-based host generator."""
    import torch
    import paper_2506_10401_b200 as hct
    from workloads import sweep
    pk = peaks()
    dev = f"cuda:{device}"
    flush = torch.empty(192 * 1024 * 1024, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(device)
    records = []
    launches = 0
    for e in sweep.entries():
        spec, laws, meta = sweep.get(e["seed"])
        gen = torch.Generator(device=dev)
        gen.manual_seed(1000 + e["seed"])
        ins = []
        for name, dtype, shape in configs.parse_inputs(spec):
            law = laws[name]
            if law["kind"] == "normal":
                t = torch.randn(shape, device=dev, generator=gen) * law.get("std", 1.0) + law.get("mean", 0.0)
            else:
                t = torch.rand(shape, device=dev, generator=gen) * (law["hi"] - law["lo"]) + law["lo"]
            ins.append(t.to(torch.bfloat16) if dtype == "bf16" else t)
        g = hct.FusedGraph.autotuned(spec, ins, device, max_trials=tune) if tune > 0 else hct.FusedGraph(spec, device)
        outs = g.alloc_outputs()
        for _ in range(max(1, warmup)):
            g.run(ins, outs, stream)
        torch.cuda.synchronize(device)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush.zero_()
            a.record(stream)
            g.run(ins, outs, stream)
            b.record(stream)
        torch.cuda.synchronize(device)
        g.status()
        sec = float(np.median([a.elapsed_time(b) for a, b in ev])) * 1e-3
        bytes_, flops = g.cost()
        t_mem = bytes_ / (pk["hbm"] * 1e9)
        t_mma = flops / (pk["tensor"] / 6.0 * 1e12)  # fp32 GEMM = three TF32 products at half the bf16 rate
        cls = "gemm" if t_mma > t_mem else "memory"
        records.append(dict(seed=e["seed"], cls=cls, us=sec * 1e6, bytes=bytes_, flops=flops, kernels=g.num_kernels, schedule=g.schedule,
                            frac=max(t_mem, t_mma) / sec))
        launches += g.num_kernels * (steps + max(1, warmup))
        g.close()
        del ins, outs
    if out_path:
        with open(out_path, "w") as f:
            for r in records:
                f.write(json.dumps(r) + "\n")
    mem = [r for r in records if r["cls"] == "memory"]
    mma = [r for r in records if r["cls"] == "gemm"]
    geo = lambda rs: float(np.exp(np.mean(np.log([r["frac"] for r in rs])))) if rs else None
    agg = dict(graphs=len(records), memory_graphs=len(mem), gemm_graphs=len(mma),
               memory_GBps=sum(r["bytes"] for r in mem) / sum(r["us"] for r in mem) / 1e3 if mem else None,
               gemm_TFLOPps_fp32=sum(r["flops"] for r in mma) / sum(r["us"] for r in mma) / 1e6 if mma else None,
               memory_frac_geomean=geo(mem), gemm_frac_geomean=geo(mma),
               memory_share_ge_0p7=float(np.mean([r["frac"] >= 0.7 for r in mem])) if mem else None,
               gemm_share_ge_0p6=float(np.mean([r["frac"] >= 0.6 for r in mma])) if mma else None,
               total_ms=sum(r["us"] for r in records) / 1e3)
    return agg, launches


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="hct", choices=["hct", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=list(WORKLOADS) + ["c5_sweep"])
    ap.add_argument("--out", default=None, help="c5_sweep: write one JSON record per graph to this file")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tune", type=int, default=0, help="pick each graph's schedule by measuring up to N candidates (untimed set-up)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    name = args.workload
    info = WORKLOADS.get(name)
    metric = "fused-chain throughput: GB/s (memory-bound) / TFLOP/s (GEMM,conv) and % of B200 roofline"

    if args.impl == "reference":
        if rank != 0:
            return
        if name == "c5_sweep":
            name = HEADLINE
        r = oracle_arm(name, max(1, min(args.steps, 5)), min(args.warmup, 1))
        line = dict(impl="reference", metric=metric, value=r["value"], unit=r["unit"], n_gpus=args.gpus, steps=args.steps,
                    warmup=args.warmup, ms_per_step=r["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="f64", data="synthetic", config={"workload": name, "sample": r["sample"]},
                    cpu_baseline=dict(value=r["value"], unit=r["unit"], cores=r["cores"], kind="oracle", sample=r["sample"]),
                    e2e=dict(value=r["value"], unit=r["unit"], h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
        print(json.dumps(line))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fused chains have no CPU execution path")
    if rank == 0:
        from paper_2506_10401_b200 import build as _build
        _build.build()  # in-tree library, rebuilt only when missing or stale
    if name == "c5_sweep":
        if world > 1:
            raise SystemExit("the sweep runs on one GPU")
        with ClockSampler(local) as clocks:
            agg, launches = run_sweep(max(3, min(args.steps, 10)), args.warmup, local, args.out, args.tune)
        pk = peaks()
        print(json.dumps(dict(metric=metric, value=agg["memory_GBps"], unit="GB/s", n_gpus=1, steps=args.steps, warmup=args.warmup,
                              ms_per_step=agg["total_ms"], higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f32",
                              data="synthetic", config={"workload": "c5_sweep: 200 random operator DAGs, seeds 0..199",
                                                        "l2": "flushed between runs", "value_is": "aggregate over memory-bound graphs",
                                                        "tuned_trials": args.tune},
                              clocks=clocks.summary(), gpu_launches=launches, sweep=agg,
                              roofline=dict(bound="hbm", achieved=agg["memory_GBps"], peak=pk["hbm"], unit="GB/s",
                                            frac=agg["memory_GBps"] / pk["hbm"], traffic=None, peak_source=pk["source"]),
                              e2e=None, cpu_baseline=None)))
        return
    if world > 1:
        torch.cuda.set_device(local)
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    r = run_gpu(name, args.steps, args.warmup, rank, world, local, args.tune)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        o = oracle_arm(name, 4, 1)
        cpu = dict(value=o["value"], unit=o["unit"], cores=o["cores"], kind="oracle", sample=o["sample"])
    if rank == 0:
        pk = peaks()
        achieved, unit = metric_of(info["bound"], r["bytes"], r["flops"], r["kernel_s"])
        # a contraction timed over a long run sits under the power cap: compare with the sustained GEMM
        # figure then, with the burst figure when the clocks stayed at their maximum
        clk = r["clocks"]
        capped = "sw_power_cap" in clk["reasons"] and clk["sm_mhz"] and clk["sm_max_mhz"] and clk["sm_mhz"] < 0.9 * clk["sm_max_mhz"]
        peak_kind = "copy" if info["bound"] == "hbm" else ("gemm sustained" if capped else "gemm burst")
        peak = pk["hbm"] if info["bound"] == "hbm" else (pk["tensor_sustained"] if capped else pk["tensor"])
        line = dict(metric=metric, value=r["value"], unit=r["unit"], n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                    ms_per_step=r["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="bf16" if ("bf16" in name or name in ("matmul_dropout_mean_softmax", "conv_block", "dwconv_bn_relu", "mbconv_block")) else "f32", data="synthetic",
                    config={"workload": name, "l2": "flushed between steps (192 MB write, untimed)", "kernels_per_step": r["kernels"],
                            "parallelism": "replicas" if world > 1 else "single",
                            "schedule": r["schedule"] or "default", "tuned_trials": args.tune},
                    clocks=r["clocks"], e2e=r["e2e"], gpu_launches=r["kernels"] * args.steps,
                    roofline=dict(bound=info["bound"], achieved=achieved, peak=peak, unit=("GB/s" if info["bound"] == "hbm" else "TFLOP/s"),
                                  frac=achieved / peak, traffic=recorded_traffic(name, r["fingerprint"]), peak_source=pk["source"],
                                  peak_kind=peak_kind, kernel_fingerprint=r["fingerprint"]),
                    cpu_baseline=cpu)
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
