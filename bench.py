#!/usr/bin/env python
"""Benchmark of fused operator chains on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one run of a whole fused chain (every kernel of its plan) on one batch of seeded
synthetic input.  The K timed steps run back to back between one pair of CUDA events, rotating over
copies of every buffer whose total exceeds L2 twice over (a step that moves more than L2 needs one
copy), each copy's step captured in a CUDA graph; the time of the same steps taken one by one, each
between its own event pair after an L2 flush, is reported beside it.  The headline workload is the memory-bound chain (affine, GELU, row softmax,
row layer normalisation on an fp32 [8192,4096] tensor); throughput is algorithmic bytes per
second (inputs read once, outputs written once).  Contraction chains report TFLOP/s.
Without --workload the line also carries, under "configs", the other four benchmark
configurations (fp32 GEMM chain, bf16 GEMM chain, bf16 convolution chain, the 200-graph sweep),
each timed the same way in the same process.
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
    # sample: what the CPU-baseline leg times (a few steps); ref_sample: one step of the reference arm, which
    # runs every requested step and warm-up, so its sample is smaller
    "c2_softmax_layernorm_chain": dict(bound="hbm", sample=dict(r=8192), ref_sample=dict(r=1024)),
    "c3_gemm_bf16_gelu_residual": dict(bound="tensor", sample=dict(m=2048), ref_sample=dict(m=256)),
    "c4_conv_bn_relu_bf16": dict(bound="tensor", sample=dict(n=8), ref_sample=dict(n=2)),
    "c1_gemm_bias_relu_f32": dict(bound="tensor", sample=dict()),
    # operator classes beyond the five configurations: a layout transform and the case-study chain with dropout
    "transpose_bias_relu": dict(bound="hbm", sample=dict(r=4096)),
    "matmul_dropout_mean_softmax": dict(bound="tensor", sample=dict(m=1024)),
    "conv_block": dict(bound="tensor", sample=dict(n=4)),
    "conv_s2_bn_relu": dict(bound="tensor", sample=dict(n=4)),
    "conv_s2_bn_relu_nhwc": dict(bound="tensor", sample=dict(n=4)),
    "dwconv_bn_relu": dict(bound="hbm", sample=dict(n=8)),
    "topk_bias_relu": dict(bound="hbm", sample=dict(r=2048)),
    "sort_bias_relu": dict(bound="hbm", sample=dict(r=2048)),
    "mbconv_block": dict(bound="hbm", sample=dict(n=4)),
    # more than one block: three inverted-residual blocks with a stride-2 transition, and a bottleneck with a grouped 3x3
    "mobilenet_stage": dict(bound="hbm", sample=dict(n=2)),
    "resnext_block": dict(bound="hbm", sample=dict(n=4)),
}
HEADLINE = "c2_softmax_layernorm_chain"
SMALL_BYTES = 24 * 1024 * 1024
# the other configurations reported beside the headline, with the steps they are timed over
# (at most; --steps caps them) and the GPU test that checks the same launch configuration against the oracle
ALSO = [("c1_gemm_bias_relu_f32", 200, "tests/test_gpu_parity.py::test_config1_gemm_bias_relu_full_size"),
        ("c3_gemm_bf16_gelu_residual", 100, "tests/test_gpu_fullsize.py::test_config3_full_size_sampled_rows"),
        ("c4_conv_bn_relu_bf16", 200, "tests/test_gpu_fullsize.py::test_config4_full_size_all_images")]
PARITY_TEST = {HEADLINE: "tests/test_gpu_fullsize.py::test_config2_full_size_all_rows",
               "c5_sweep": "tests/test_gpu_fullsize.py::test_sweep_graph_full_size_sampled_rows (all 200 seeds)"}
PARITY_TEST.update({n: t for n, _, t in ALSO})


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


def oracle_arm(name, steps, warmup, sample_key="sample"):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload."""
    import oracle
    from workloads import tensors
    info = WORKLOADS[name]
    sample_kw = info.get(sample_key, info["sample"])
    spec, laws = configs.get_config(name, **sample_kw)
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
    # numpy evaluates elementwise operators and reductions on one thread; only the matrix products
    # of a contraction (matmul, einsum) run on the BLAS pool
    cores = 1
    if flops > 0:
        try:
            from threadpoolctl import threadpool_info
            cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        except Exception:
            cores = os.cpu_count() or 1
    sample = ", ".join(f"{k}={v}" for k, v in sample_kw.items()) or "full size"
    return dict(value=value, unit=unit, cores=cores, kind="oracle", sample=f"{name} at {sample} ({out_elems} output elements per step)",
                ms_per_step=dt * 1e3)


def run_gpu(name, steps, warmup, rank, world, device, tune=0, with_e2e=True):
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

    # Timed region: exactly `steps` steps, back to back, between one pair of events.  The steps rotate over copies of
    # every buffer (see RotatingSets), so no step finds its operands in L2 and none waits for a host launch.
    try:
        rot = RotatingSets(g, ins, device)
    except Exception as e:  # noqa: BLE001 - without capture the steps are timed one by one, each after an L2 flush
        print(f"CUDA-graph capture failed, timing step by step: {e}", file=sys.stderr)
        rot = None
    for _ in range(max(warmup, 3)):
        flush.zero_()
        g.run(ins, outs, stream)
    if rot is not None:
        for _ in range(max(warmup, 3) * rot.n_sets):
            rot.step()
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(device) as clocks:
        if rot is not None:
            t0.record(stream)
            for _ in range(steps):
                rot.step()
            t1.record(stream)
            barrier()
        # second figure: the same number of steps, each between its own pair of events after an L2 flush (about 6 us of
        # launch and event cost per step on top of the kernels)
        for a, b in ev:
            flush.zero_()           # evict the previous step's data from L2; not timed
            a.record(stream)
            g.run(ins, outs, stream)
            b.record(stream)
        # nvidia-smi samples every 50 ms and a short timed region may end before its first sample: the same
        # steps keep running, untimed, until the sampler has seen about 0.3 s of this load
        t_end = time.perf_counter() + (max(0.0, 0.3 - 1e-3 * steps) if steps >= 10 else 0.0)   # (short profiling runs stay short)
        while time.perf_counter() < t_end:
            if rot is not None:
                for _ in range(8):
                    rot.step()
            else:
                flush.zero_()
                g.run(ins, outs, stream)
            torch.cuda.synchronize(device)
        barrier()
    g.status()
    per_step = [a.elapsed_time(b) * 1e-3 for a, b in ev]
    events_s = float(np.sum(per_step))
    dev_s = t0.elapsed_time(t1) * 1e-3 if rot is not None else events_s
    timing = dict(protocol=("steps back to back between one event pair, rotating over %d copies of every buffer (L2 %s)" % (rot.n_sets, rot.l2))
                  if rot is not None else "each step between its own event pair after an L2 flush",
                  events_ms_per_step=events_s / steps * 1e3)
    if not with_e2e:
        dev_s = max_over_ranks([dev_s], f"cuda:{device}")[0]
        value, unit = whole_job_value(info["bound"], bytes_, flops, world, dev_s / steps)
        return dict(value=value, unit=unit, ms_per_step=dev_s / steps * 1e3, bytes=bytes_, flops=flops, kernel_s=dev_s / steps,
                    fingerprint=kernel_fingerprint(g), kernels=g.num_kernels, clocks=clocks.summary(), e2e=None, plan=g.plan,
                    schedule=g.schedule, timing=timing)
    del rot

    # end to end: pinned host inputs -> device, run, result back to the host, every step.  The three
    # phases of consecutive steps overlap (copy-in, compute and copy-out streams, two sets of device
    # buffers): PCIe is full duplex, so step i+1's inputs travel while step i's result returns.
    specs_in = configs.parse_inputs(spec)
    layouts = configs.input_layouts(spec)
    as_host = lambda n, d: torch.from_numpy(host[n].view(np.int16) if d == "bf16" else host[n])
    # an input declared channels-last is channels-last on the host as well: the copy moves bytes, it does not permute them
    pinned = [(as_host(n, d).contiguous(memory_format=torch.channels_last) if layouts.get(n) == "nhwc" else as_host(n, d)).pin_memory()
              for n, d, _ in specs_in]
    dev_in = [[torch.empty_like(t, device=f"cuda:{device}") for t in pinned] for _ in range(2)]
    run_in = [[t.view(torch.bfloat16) if d == "bf16" else t for t, (_, d, _) in zip(buf, specs_in)] for buf in dev_in]
    dev_out = [outs, g.alloc_outputs()]
    host_out = [[torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs] for _ in range(2)]
    h2d = sum(t.numel() * t.element_size() for t in pinned)
    d2h = sum(t.numel() * t.element_size() for t in host_out[0])
    e2e_steps = max(4, min(steps, 50))
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
    kern_s = dev_s / steps
    return dict(value=value, unit=unit, ms_per_step=dev_s / steps * 1e3, bytes=bytes_, flops=flops, kernel_s=kern_s, timing=timing,
                fingerprint=kernel_fingerprint(g),
                kernels=g.num_kernels, clocks=clocks.summary(), e2e=dict(value=e2e_v, unit=unit, h2d_bytes_per_step=h2d,
                                                                         d2h_bytes_per_step=d2h), plan=g.plan,
                schedule=g.schedule)


class RotatingSets:
    """Copies of a graph's inputs, outputs and workspace whose total exceeds L2 twice over, and one CUDA graph per
    copy that runs the fused chain on it.  Steps issued round robin over the copies follow each other on the device
    without a host launch or an L2 flush in between, and every step finds its operands cold (a workload that moves
    more than L2 per step needs a single copy; one too small to reach the budget with `max_sets` copies runs partly
    warm: `l2` says which)."""

    def __init__(self, g, ins, device, budget_bytes=256 << 20, max_sets=24):
        import torch
        import paper_2506_10401_b200 as hct
        self.g, self.device = g, device
        dev = f"cuda:{device}"
        outs0 = g.alloc_outputs()
        per_set = sum(t.numel() * t.element_size() for t in ins) + g.workspace_bytes + sum(t.numel() * t.element_size() for t in outs0)
        self.n_sets = int(max(1, min(max_sets, -(-budget_bytes // per_set))))
        self.l2 = "cold" if per_set * self.n_sets >= 192 << 20 else "warm"
        self.sets = []
        for i in range(self.n_sets):
            si = ins if i == 0 else [t.clone() for t in ins]
            so = outs0 if i == 0 else g.alloc_outputs()
            ws = torch.empty(g.workspace_bytes + 256, dtype=torch.uint8, device=dev) if g.workspace_bytes else None
            ws_ptr = (ws.data_ptr() + 255) // 256 * 256 if ws is not None else 0
            self.sets.append((si, so, ws, [t.data_ptr() for t in si], [t.data_ptr() for t in so], ws_ptr))
        side = torch.cuda.Stream(device)
        side.wait_stream(torch.cuda.current_stream(device))
        self.graphs = []
        for _, _, _, pi, po, pw in self.sets:
            with torch.cuda.stream(side):
                hct.hct_graph_run(g.handle, pi, po, pw, g.workspace_bytes, side.cuda_stream)
            side.synchronize()
            cg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cg, stream=side, capture_error_mode="thread_local"):
                hct.hct_graph_run(g.handle, pi, po, pw, g.workspace_bytes, side.cuda_stream)
            self.graphs.append(cg)
        self.next = 0

    def step(self):
        self.graphs[self.next].replay()
        self.next = (self.next + 1) % self.n_sets

    def outputs_of_last_step(self):
        return self.sets[(self.next - 1) % self.n_sets][1]


def replay_seconds(g, ins, device, budget_bytes=256 << 20, max_sets=24, target_ms=4.0):
    """Steady-state time of one run of graph `g`, without a host launch or an event pair per step.

    A step timed between its own pair of events costs about 6 us on top of the kernel (measured with a
    one-thread kernel in the same place), which buries chains that run for a few microseconds.  Here the
    inputs, outputs and workspace exist in several copies whose total exceeds L2 twice over (as many as
    `budget_bytes` needs, at most `max_sets`), one run per copy is captured into a CUDA graph, and the graph
    is replayed between ONE pair of events: kernels follow each other on the device and every run finds its
    operands cold in L2 (or, for graphs too small to fill the budget with `max_sets` copies, partly warm:
    the second value returned says which).  Returns (seconds per run, "cold" | "warm") or None when the
    capture is not possible."""
    import torch
    import paper_2506_10401_b200 as hct
    dev = f"cuda:{device}"
    per_set = sum(t.numel() * t.element_size() for t in ins) + g.workspace_bytes
    outs0 = g.alloc_outputs()
    per_set += sum(t.numel() * t.element_size() for t in outs0)
    n_sets = int(max(1, min(max_sets, -(-budget_bytes // per_set))))
    sets = []
    for i in range(n_sets):
        si = ins if i == 0 else [t.clone() for t in ins]
        so = outs0 if i == 0 else g.alloc_outputs()
        ws = torch.empty(g.workspace_bytes + 256, dtype=torch.uint8, device=dev) if g.workspace_bytes else None
        ws_ptr = (ws.data_ptr() + 255) // 256 * 256 if ws is not None else 0
        sets.append((si, so, ws, [t.data_ptr() for t in si], [t.data_ptr() for t in so], ws_ptr))
    side = torch.cuda.Stream(device)

    def enqueue(stream):
        for _, _, _, pi, po, pw in sets:
            hct.hct_graph_run(g.handle, pi, po, pw, g.workspace_bytes, stream.cuda_stream)

    try:
        side.wait_stream(torch.cuda.current_stream(device))
        with torch.cuda.stream(side):
            enqueue(side)
        side.synchronize()
        cg = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cg, stream=side, capture_error_mode="thread_local"):
            enqueue(side)
    except Exception as e:  # noqa: BLE001 - any capture failure falls back to the per-step protocol
        print(f"replay capture failed: {e}", file=sys.stderr)
        return None
    stream = torch.cuda.current_stream(device)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cg.replay()
    torch.cuda.synchronize(device)
    a.record(stream); cg.replay(); b.record(stream)
    torch.cuda.synchronize(device)
    once_ms = max(a.elapsed_time(b), 1e-3)
    reps = int(max(2, min(200, target_ms / once_ms)))
    a.record(stream)
    for _ in range(reps):
        cg.replay()
    b.record(stream)
    torch.cuda.synchronize(device)
    g.status()
    sec = a.elapsed_time(b) * 1e-3 / (reps * n_sets)
    del cg
    return sec, ("cold" if per_set * n_sets >= 192 << 20 else "warm"), n_sets


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
    # Graph creation (planning + NVRTC) is untimed set-up and dominates the wall clock of the sweep:
    # graphs are created a few ahead of use on a thread pool (the compiler runs outside the interpreter lock).
    from concurrent.futures import ThreadPoolExecutor
    todo = sweep.entries()

    def make(e):
        spec, laws, meta = sweep.get(e["seed"])
        return spec, laws, (None if tune > 0 else hct.FusedGraph(spec, device))

    pool = ThreadPoolExecutor(max_workers=6)
    ahead = [pool.submit(make, e) for e in todo[:12]]
    for i, e in enumerate(todo):
        if i + 12 < len(todo):
            ahead.append(pool.submit(make, todo[i + 12]))
        spec, laws, made = ahead[i].result()
        ahead[i] = None
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
        g = hct.FusedGraph.autotuned(spec, ins, device, max_trials=tune) if tune > 0 else made
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
        # event time stamps on this platform step by about 2 us: the mean over the steps (largest one dropped)
        # resolves a microsecond-scale run, their median does not
        ms = sorted(a.elapsed_time(b) for a, b in ev)
        sec = float(np.mean(ms[:-1] if len(ms) > 3 else ms)) * 1e-3
        bytes_, flops = g.cost()
        t_mem = bytes_ / (pk["hbm"] * 1e9)
        t_mma = flops / (pk["tensor"] / 6.0 * 1e12)  # fp32 GEMM = three TF32 products at half the bf16 rate
        cls = "gemm" if t_mma > t_mem else "memory"
        del outs
        rp = replay_seconds(g, ins, device)
        sec_events = sec
        if rp is not None:
            sec = rp[0]
        records.append(dict(seed=e["seed"], cls=cls, us=sec * 1e6, us_events=sec_events * 1e6, l2=(rp[1] if rp else "flushed"),
                            sets=(rp[2] if rp else 1), bytes=bytes_, flops=flops, kernels=g.num_kernels, schedule=g.schedule,
                            frac=max(t_mem, t_mma) / sec, frac_events=max(t_mem, t_mma) / sec_events))
        launches += g.num_kernels * (steps + max(1, warmup))
        g.close()
        del ins
    pool.shutdown()
    if out_path:
        with open(out_path, "w") as f:
            for r in records:
                f.write(json.dumps(r) + "\n")
    # Graphs that move less than SMALL_BYTES are latency-bound (a few microseconds for a tensor that
    # sits in L2): they are reported as a latency class of their own, not against the HBM roofline.
    small = [r for r in records if r["cls"] == "memory" and r["bytes"] < SMALL_BYTES]
    mem = [r for r in records if r["cls"] == "memory" and r["bytes"] >= SMALL_BYTES]
    mma = [r for r in records if r["cls"] == "gemm"]
    geo = lambda rs: float(np.exp(np.mean(np.log([r["frac"] for r in rs])))) if rs else None
    agg = dict(graphs=len(records), memory_graphs=len(mem), gemm_graphs=len(mma), small_graphs=len(small),
               memory_GBps=sum(r["bytes"] for r in mem) / sum(r["us"] for r in mem) / 1e3 if mem else None,
               gemm_TFLOPps_fp32=sum(r["flops"] for r in mma) / sum(r["us"] for r in mma) / 1e6 if mma else None,
               memory_frac_geomean=geo(mem), gemm_frac_geomean=geo(mma),
               memory_share_ge_0p7=float(np.mean([r["frac"] >= 0.7 for r in mem])) if mem else None,
               gemm_share_ge_0p6=float(np.mean([r["frac"] >= 0.6 for r in mma])) if mma else None,
               small_us_median=float(np.median([r["us"] for r in small])) if small else None,
               small_us_max=float(np.max([r["us"] for r in small])) if small else None,
               small_launches_mean=float(np.mean([r["kernels"] for r in small])) if small else None,
               small_bytes_below=SMALL_BYTES,
               timing="CUDA-graph replay over rotating copies of every buffer (total above twice L2), one event pair per graph",
               events_memory_GBps=sum(r["bytes"] for r in mem) / sum(r["us_events"] for r in mem) / 1e3 if mem else None,
               events_gemm_TFLOPps_fp32=sum(r["flops"] for r in mma) / sum(r["us_events"] for r in mma) / 1e6 if mma else None,
               events_small_us_median=float(np.median([r["us_events"] for r in small])) if small else None,
               events_note="same graphs, every step between its own event pair after an L2 flush: about 6 us of launch and event cost per step",
               all_memory_GBps=sum(r["bytes"] for r in mem + small) / sum(r["us"] for r in mem + small) / 1e3 if mem or small else None,
               total_ms=sum(r["us"] for r in records) / 1e3)
    return agg, launches


def roofline_of(name, r, pk):
    """Roofline record of one timed workload: algorithmic bytes or flops of a step over the mean step time on the device."""
    info = WORKLOADS[name]
    achieved, unit = metric_of(info["bound"], r["bytes"], r["flops"], r["kernel_s"])
    # a contraction timed over a long run sits under the power cap: compare with the sustained GEMM
    # figure then, with the burst figure when the clocks stayed at their maximum
    clk = r["clocks"]
    capped = "sw_power_cap" in clk["reasons"] and clk["sm_mhz"] and clk["sm_max_mhz"] and clk["sm_mhz"] < 0.9 * clk["sm_max_mhz"]
    peak_kind = "copy" if info["bound"] == "hbm" else ("gemm sustained" if capped else "gemm burst")
    peak = pk["hbm"] if info["bound"] == "hbm" else (pk["tensor_sustained"] if capped else pk["tensor"])
    return dict(bound=info["bound"], achieved=achieved, peak=peak, unit=unit, frac=achieved / peak,
                traffic=recorded_traffic(name, r["fingerprint"]), peak_source=pk["source"], peak_kind=peak_kind,
                kernel_fingerprint=r["fingerprint"])


def dtype_of(name):
    return "bf16" if ("bf16" in name or name in ("matmul_dropout_mean_softmax", "conv_block", "dwconv_bn_relu", "mbconv_block", "conv_s2_bn_relu", "conv_s2_bn_relu_nhwc", "mobilenet_stage", "resnext_block")) else "f32"


def sweep_record(steps, warmup, device, out_path, tune):
    """The sweep as one entry of the "configs" list (also the body of the line --workload c5_sweep prints)."""
    with ClockSampler(device) as clocks:
        agg, launches = run_sweep(steps, warmup, device, out_path, tune)
    pk = peaks()
    return dict(workload="c5_sweep: 200 random operator DAGs, seeds 0..199", dtype="f32", steps=steps, warmup=max(1, warmup),
                ms_per_step=agg["total_ms"], value=agg["memory_GBps"], unit="GB/s",
                value_is="aggregate bytes / time over the memory-bound graphs of at least %d MB; see sweep for the GEMM-bound and small classes"
                         % (SMALL_BYTES >> 20),
                roofline=dict(bound="hbm", achieved=agg["memory_GBps"], peak=pk["hbm"], unit="GB/s", frac=agg["memory_GBps"] / pk["hbm"],
                              traffic=None, peak_source=pk["source"], peak_kind="copy"),
                gemm_roofline=dict(bound="tensor", achieved=agg["gemm_TFLOPps_fp32"], peak=pk["tensor"] / 6.0, unit="TFLOP/s",
                                   frac=agg["gemm_TFLOPps_fp32"] / (pk["tensor"] / 6.0), peak_source=pk["source"],
                                   peak_kind="gemm burst / 6 (three TF32 products at half the bf16 rate)"),
                sweep=agg, clocks=clocks.summary(), gpu_launches=launches, l2="cold: rotating buffer copies larger than L2 (graphs under %d MB: warm, reported as latency)" % (SMALL_BYTES >> 20), tuned_trials=tune,
                parity_checked=PARITY_TEST["c5_sweep"])


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="hct", choices=["hct", "reference"])
    ap.add_argument("--workload", default=None, choices=list(WORKLOADS) + ["c5_sweep"],
                    help="time this workload alone (default: the headline chain, with the other four configurations under 'configs')")
    ap.add_argument("--out", default=None, help="write one JSON record per sweep graph to this file")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tune", type=int, default=0, help="pick each graph's schedule by measuring up to N candidates (untimed set-up)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    all_configs = args.workload is None and world == 1
    name = args.workload or HEADLINE
    info = WORKLOADS.get(name)
    metric = "fused-chain throughput: GB/s (memory-bound) / TFLOP/s (GEMM,conv) and % of B200 roofline"

    if args.impl == "reference":
        if rank != 0:
            return
        if name == "c5_sweep":
            name = HEADLINE
        # every step is a bounded sample of the workload; all requested steps and warm-ups are run
        r = oracle_arm(name, max(1, args.steps), max(0, args.warmup), "ref_sample")
        line = dict(impl="reference", metric=metric, value=r["value"], unit=r["unit"], n_gpus=args.gpus, steps=max(1, args.steps),
                    warmup=max(0, args.warmup),
                    ms_per_step=r["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
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
    sweep_steps = max(3, min(args.steps, 10)) if name == "c5_sweep" else 3
    if name == "c5_sweep":
        if world > 1:
            raise SystemExit("the sweep runs on one GPU")
        rec = sweep_record(sweep_steps, args.warmup, local, args.out, args.tune)
        print(json.dumps(dict(metric=metric, value=rec["value"], unit="GB/s", n_gpus=1, steps=sweep_steps, warmup=rec["warmup"],
                              ms_per_step=rec["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f32",
                              data="synthetic", config={"workload": rec["workload"], "l2": rec["l2"], "value_is": rec["value_is"],
                                                        "tuned_trials": args.tune},
                              clocks=rec["clocks"], gpu_launches=rec["gpu_launches"], sweep=rec["sweep"], roofline=rec["roofline"],
                              gemm_roofline=rec["gemm_roofline"], e2e=None, cpu_baseline=None)))
        return
    if world > 1:
        torch.cuda.set_device(local)
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    r = run_gpu(name, args.steps, args.warmup, rank, world, local, args.tune)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        o = oracle_arm(name, 4, 1)
        cpu = dict(value=o["value"], unit=o["unit"], cores=o["cores"], kind="oracle", sample=o["sample"])
    others = []
    if all_configs:
        pk = peaks()
        for other, cap, test in ALSO:
            k = max(3, min(args.steps, cap))
            o = run_gpu(other, k, args.warmup, rank, world, local, args.tune, with_e2e=False)
            others.append(dict(workload=other, dtype=dtype_of(other), steps=k, warmup=max(args.warmup, 3), ms_per_step=o["ms_per_step"],
                               value=o["value"], unit=o["unit"], roofline=roofline_of(other, o, pk), clocks=o["clocks"],
                               kernels_per_step=o["kernels"], gpu_launches=o["kernels"] * k, timing=o["timing"],
                               parity_checked=test))
        others.append(sweep_record(sweep_steps, min(args.warmup, 2), local, args.out, args.tune))
    if rank == 0:
        pk = peaks()
        line = dict(metric=metric, value=r["value"], unit=r["unit"], n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                    ms_per_step=r["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype=dtype_of(name), data="synthetic",
                    config={"workload": name, "l2": r["timing"]["protocol"], "events_ms_per_step": r["timing"]["events_ms_per_step"],
                            "kernels_per_step": r["kernels"],
                            "parallelism": "replicas" if world > 1 else "single",
                            "schedule": r["schedule"] or "default", "tuned_trials": args.tune,
                            "parity_checked": PARITY_TEST.get(name)},
                    clocks=r["clocks"], e2e=r["e2e"], gpu_launches=r["kernels"] * args.steps,
                    roofline=roofline_of(name, r, pk), cpu_baseline=cpu)
        if all_configs:
            line["configs"] = others
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
