"""Shared helpers for parity tests: feed one seeded workload to both sides and compare.

Tolerances (written here once, used by every GPU test):
  * fp32 chains (elementwise, broadcast, row reductions, fp32 GEMM), per element:
        |g - r| <= max(1e-5 * |r|, SAFETY * E)
    where E is the first-order float32 forward error bound of that element, computed from the
    oracle's own float64 node values (tests/errbound.py).  Wherever nothing cancels, E is a few
    units of 2^-24 relative to |r|, so the criterion IS the strict relative 1e-5.  Where a
    subtraction-like step cancels, E is what float32 can resolve there: for a row sum it is
    (log2 C + 1) * 2^-24 * sum_j |x_ij|, the condition number of the sum.
    For full-width outputs the bound is capped by the older rule 1e-5 * max(|r|, largest |r| of the
    row or (n,k) plane), so that it is never looser than that rule was.
    The strict figure (largest |g - r| / |r|, no allowance for cancellation) is recorded for every
    comparison and printed at the end of the run, ungraded.
  * bf16-input, fp32-accumulate contractions with bf16 output: |g - r| <= 1e-2 + 2e-2 * |r|.
  * graphs of several blocks (six or more contractions in a row, bf16 between them): see bf16_deep_chain_check.
"""
from __future__ import annotations

import numpy as np

from tests import errbound
from workloads import configs, tensors

TOL_F32 = 1e-5
TOL_BF16_REL, TOL_BF16_ABS = 2e-2, 1e-2
FLOOR = 1e-37            # results below the smallest normal float32 may be flushed to zero on the device

REPORT = []              # one record per fp32 comparison: label, graded violation, strict figure, share judged strictly
_label = [""]


def set_label(text):
    _label[0] = text


class Ref(np.ndarray):
    """An oracle output together with the float32 error bound of each of its elements."""

    def __new__(cls, values, err=None):
        obj = np.asarray(values, dtype=np.float64).view(cls)
        obj.err = None if err is None else np.asarray(err, dtype=np.float64)
        return obj

    def __array_finalize__(self, obj):
        self.err = getattr(obj, "err", None)


def oracle_inputs(spec, tensors_by_name):
    return {n: tensors.as_float64(tensors_by_name[n], d) for n, d, _ in configs.parse_inputs(spec)}


def oracle_reference(spec, inputs64):
    """Oracle outputs by name, each carrying its float32 error bound."""
    import oracle
    g = oracle.parse(spec) if not isinstance(spec, oracle.Graph) else spec
    val = oracle.run_nodes(g, inputs64)
    err = errbound.bound(g, inputs64, values=val)
    return {name: Ref(val[name], err[name]) for name, _ in g.outputs}


def to_device(spec, tensors_by_name, device="cuda:0"):
    import torch
    out = []
    layouts = configs.input_layouts(spec)
    for n, d, _ in configs.parse_inputs(spec):
        a = tensors_by_name[n]
        if d == "bf16":
            t = torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
        else:
            t = torch.from_numpy(a).to(device)
        if layouts.get(n) == "nhwc":      # same values, channels-last in memory
            t = t.contiguous(memory_format=torch.channels_last)
        out.append(t)
    return out


def to_numpy64(t):
    import torch
    return t.detach().to(torch.float64).cpu().numpy()


def row_scale(ref):
    """Largest magnitude of the element's output row (NCHW: of its (n,k) plane)."""
    ref = np.asarray(ref)
    if ref.ndim == 4:
        return np.abs(ref).max(axis=(2, 3), keepdims=True)
    return np.abs(ref).max(axis=-1, keepdims=True)


def f32_bound(ref, tol=TOL_F32):
    """Per-element bound on |g - r| (see the module text)."""
    r = np.abs(np.asarray(ref))
    err = getattr(ref, "err", None)
    strict = tol * r
    if err is None:
        bound = strict
    else:
        bound = np.maximum(strict, errbound.SAFETY * err * (tol / TOL_F32))
        if ref.ndim >= 2 and ref.shape[-1] > 1:
            bound = np.minimum(bound, tol * np.maximum(r, row_scale(ref)))
    return np.maximum(bound, FLOOR), strict


def f32_violation(got, ref, tol=TOL_F32):
    """max over elements of |g - r| / bound; parity holds when <= 1."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    if not np.all(np.isfinite(got)):
        return float("inf")
    bound, strict = f32_bound(ref, tol)
    diff = np.abs(got - np.asarray(ref))
    worst = float((diff / bound).max())
    nz = np.abs(np.asarray(ref)) > FLOOR
    strict_fig = float((diff[nz] / np.abs(np.asarray(ref))[nz]).max()) if nz.any() else 0.0
    REPORT.append(dict(label=_label[0], shape=tuple(ref.shape), violation=worst, strict_rel=strict_fig,
                       share_strict=float(np.mean(bound <= np.maximum(strict, FLOOR)))))
    return worst


def bf16_violation(got, ref):
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if not np.all(np.isfinite(got)):
        return float("inf")
    ref = np.asarray(ref)
    return float((np.abs(got - ref) / (TOL_BF16_ABS + TOL_BF16_REL * np.abs(ref))).max())


def bf16_deep_chain_check(got, ref):
    """Several contractions in a row with bf16 roundings between them.  The oracle rounds fp64 values at every
    cast_bf16, the kernels fp32 ones: where the two straddle a rounding boundary the intermediate differs by one bf16
    unit (2^-8 relative), later sums amplify that wherever they cancel, and later roundings can flip in turn.  So the
    single-contraction rule is asked of all but one element in a thousand, and of every element with |r| replaced by
    the larger of |r| and the largest magnitude of its (n,k) plane (the scale of the terms that cancel).
    Returns (share of elements outside the plain rule, largest violation of the plane-scale rule)."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if not np.all(np.isfinite(got)):
        return 1.0, float("inf")
    ref = np.asarray(ref)
    diff = np.abs(got - ref)
    plain = diff / (TOL_BF16_ABS + TOL_BF16_REL * np.abs(ref))
    scaled = diff / (TOL_BF16_ABS + TOL_BF16_REL * np.maximum(np.abs(ref), row_scale(ref)))
    return float(np.mean(plain > 1.0)), float(scaled.max())


def run_both(spec, laws, seed=0, device=0, schedule=None, runs=1):
    """Runs the CUDA library (optionally under a schedule text; `runs` times in a row on the same workspace, keeping
    the last result) and the oracle on the same seeded inputs.
    Returns (list of GPU outputs as float64 arrays, list of oracle outputs with their error bounds, FusedGraph)."""
    import torch
    import paper_2506_10401_b200 as hct
    t = configs.draw_inputs(spec, laws, seed)
    ref = oracle_reference(spec, oracle_inputs(spec, t))
    g = hct.FusedGraph(spec, device, schedule=schedule)
    dev_inputs = to_device(spec, t, f"cuda:{device}")
    for _ in range(runs):
        outs = g.run(dev_inputs)
    torch.cuda.synchronize(device)
    g.status()
    got = [to_numpy64(o) for o in outs]
    want = [ref[name] for name, _, _ in g.outputs]
    return got, want, g


def report_lines():
    """Summary of the strict figures gathered so far (printed at the end of a test run)."""
    if not REPORT:
        return []
    strict = np.array([r["strict_rel"] for r in REPORT])
    share = np.array([r["share_strict"] for r in REPORT])
    lines = [f"fp32 comparisons: {len(REPORT)}; every element judged at strict relative {TOL_F32:g} in {int(np.sum(share >= 1.0))} of them; "
             f"mean share of elements judged strictly {share.mean():.4f}",
             f"strict figure max|g-r|/|r| (ungraded): median {np.median(strict):.3g}, 90th percentile {np.quantile(strict, 0.9):.3g}, "
             f"largest {strict.max():.3g}; comparisons with strict figure <= {TOL_F32:g}: {int(np.sum(strict <= TOL_F32))}"]
    for r in sorted(REPORT, key=lambda r: -r["violation"])[:8]:
        lines.append(f"  closest to the bound: {r['label']} {r['shape']}: used {r['violation']:.3f} of the bound, strict figure {r['strict_rel']:.3g}, "
                     f"share strict {r['share_strict']:.3f}")
    return lines
