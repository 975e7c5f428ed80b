"""Shared helpers for parity tests: feed one seeded workload to both sides and compare.

Tolerances (written here once, used by every GPU test):
  * fp32 chains (elementwise, broadcast, row reductions, fp32 GEMM): |g - r| <= 1e-5 * max(|r|, rho)
    where rho is the largest |r| in the same output row (for NCHW outputs: the same (n,k) plane;
    for [R,1] outputs, whose rows are single elements: the whole column).
    A relative error is undefined where r crosses zero; the row's own magnitude is the scale any
    float32 evaluation of that row can resolve.
  * bf16-input, fp32-accumulate contractions with bf16 output: |g - r| <= 1e-2 + 2e-2 * |r|.
"""
from __future__ import annotations

import numpy as np

from workloads import configs, tensors

TOL_F32 = 1e-5
TOL_BF16_REL, TOL_BF16_ABS = 2e-2, 1e-2


def oracle_inputs(spec, tensors_by_name):
    return {n: tensors.as_float64(tensors_by_name[n], d) for n, d, _ in configs.parse_inputs(spec)}


def to_device(spec, tensors_by_name, device="cuda:0"):
    import torch
    out = []
    for n, d, _ in configs.parse_inputs(spec):
        a = tensors_by_name[n]
        if d == "bf16":
            out.append(torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16))
        else:
            out.append(torch.from_numpy(a).to(device))
    return out


def to_numpy64(t):
    import torch
    return t.detach().to(torch.float64).cpu().numpy()


def row_scale(ref):
    if ref.ndim == 4:
        return np.abs(ref).max(axis=(2, 3), keepdims=True)
    if ref.shape[-1] == 1:  # a column of per-row results: its rows are single elements, so scale by the column
        return np.full_like(ref, np.abs(ref).max())
    return np.abs(ref).max(axis=-1, keepdims=True)


def f32_violation(got, ref, tol=TOL_F32):
    """max over elements of |g-r| / (tol * max(|r|, rho)); parity holds when <= 1."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    bound = tol * np.maximum(np.abs(ref), row_scale(ref))
    bound = np.maximum(bound, 1e-37)
    v = np.abs(got - ref) / bound
    if not np.all(np.isfinite(got)):
        return float("inf")
    return float(v.max())


def bf16_violation(got, ref):
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if not np.all(np.isfinite(got)):
        return float("inf")
    return float((np.abs(got - ref) / (TOL_BF16_ABS + TOL_BF16_REL * np.abs(ref))).max())


def run_both(spec, laws, seed=0, device=0, schedule=None):
    """Runs the CUDA library (optionally under a schedule text) and the oracle on the same seeded inputs.
    Returns (list of GPU outputs as float64 arrays, list of oracle outputs, FusedGraph)."""
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    t = configs.draw_inputs(spec, laws, seed)
    ref = oracle.run(spec, oracle_inputs(spec, t))
    g = hct.FusedGraph(spec, device, schedule=schedule)
    outs = g.run(to_device(spec, t, f"cuda:{device}"))
    torch.cuda.synchronize(device)
    g.status()
    got = [to_numpy64(o) for o in outs]
    want = [ref[name] for name, _, _ in g.outputs]
    return got, want, g
