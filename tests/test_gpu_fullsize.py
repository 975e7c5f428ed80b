"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Every operator is row-local (conv: image-local), so the oracle can reproduce any subset of output
rows from the matching rows of the inputs: the GPU runs the full-size graph, the oracle runs the
same spec with the sampled rows only (row-shaped inputs sliced, weights and row vectors whole),
and the sampled outputs are compared element by element."""
import numpy as np
import pytest

from tests import parity
from workloads import configs, sweep

pytestmark = pytest.mark.gpu


def _sample_rows(r, n=48):
    rng = np.random.default_rng(7)
    fixed = [0, 1, 127, 128, 129, r // 2, r - 2, r - 1]
    rows = sorted(set([x for x in fixed if 0 <= x < r] + list(rng.integers(0, r, size=n))))
    return np.array(rows)


def _run_full_and_sampled(spec_full, spec_of_rows, laws, seed, row_inputs, rows_total):
    """GPU on the full spec; oracle on spec_of_rows(len(rows)) with row-shaped inputs sliced."""
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    t = configs.draw_inputs(spec_full, laws, seed)
    g = hct.FusedGraph(spec_full, 0)
    outs = g.run(parity.to_device(spec_full, t))
    torch.cuda.synchronize()
    g.status()
    rows = _sample_rows(rows_total)
    small = {k: (v[rows] if k in row_inputs else v) for k, v in t.items()}
    spec_small = spec_of_rows(len(rows))
    ref = oracle.run(spec_small, parity.oracle_inputs(spec_small, small))
    got = [parity.to_numpy64(o[torch.from_numpy(rows).to(o.device)]) for o in outs]
    want = [ref[name] for name, _, _ in g.outputs]
    return got, want, g


def test_config2_full_size_all_rows():
    spec, laws = configs.get_config("c2_softmax_layernorm_chain")
    got, want, g = parity.run_both(spec, laws, 0)
    assert g.num_kernels == 1
    assert parity.f32_violation(got[0], want[0]) <= 1.0


def test_config3_full_size_sampled_rows():
    spec, laws = configs.get_config("c3_gemm_bf16_gelu_residual")
    got, want, g = _run_full_and_sampled(spec, lambda m: configs.get_config("c3_gemm_bf16_gelu_residual", m=m)[0], laws, 0,
                                         {"x", "r"}, 8192)
    assert "tcgen05" in g.plan
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


def test_config4_full_size_sampled_images():
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16")
    t = configs.draw_inputs(spec, laws, 0)
    g = hct.FusedGraph(spec, 0)
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    assert "tcgen05" in g.plan
    imgs = np.array([0, 13, 31])
    small = dict(t)
    small["x"] = t["x"][imgs]
    spec_small, _ = configs.get_config("c4_conv_bn_relu_bf16", n=len(imgs))
    ref = oracle.run(spec_small, parity.oracle_inputs(spec_small, small))["t3"]
    got = parity.to_numpy64(out[torch.from_numpy(imgs).to(out.device)])
    assert parity.bf16_violation(got, ref) <= 1.0


@pytest.mark.parametrize("seed", [3, 26, 55, 90, 126, 171])
def test_sweep_graph_full_size_sampled_rows(seed):
    spec, laws, meta = sweep.get(seed)
    import re
    weights = set(re.findall(r"gemm\(\w+,\s*(\w+)\)", spec))
    row_inputs = {n for n, _, s in configs.parse_inputs(spec) if len(s) == 2 and s[0] == meta["rows"] and n not in weights}
    got, want, g = _run_full_and_sampled(spec, lambda m: sweep.get(seed, rows=m)[0], laws, seed, row_inputs, meta["rows"])
    worst = max(parity.f32_violation(a, b) for a, b in zip(got, want))
    assert worst <= 1.0, f"seed {seed}: violated by factor {worst:.3g}\n{g.plan}"
