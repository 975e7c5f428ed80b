"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Every operator is row-local (conv: image-local), so the oracle can reproduce any subset of output
rows from the matching rows of the inputs: the GPU runs the full-size graph, the oracle runs the
same spec with the sampled rows only (row-shaped inputs sliced, weights and row vectors whole),
and the sampled outputs are compared element by element.

For the 200 sweep graphs and the 60 grown graphs the host generator draws the sampled rows only
(it would take minutes to draw 10^10 elements on the host): the device tensors are filled with
values of the same law drawn on the device, and the sampled rows are overwritten with the host's.
Row-locality makes the sampled output rows depend on nothing else."""
import re

import numpy as np
import pytest

from tests import parity
from workloads import configs, sweep

pytestmark = pytest.mark.gpu


def _sample_rows(r, n=40):
    rng = np.random.default_rng(7)
    # tile boundaries of the 128-row CTA tiles and the 256-row CTA-pair tiles, both ends, and the last tile's first row
    fixed = [0, 1, 127, 128, 129, 255, 256, 257, r // 2, r - 257, r - 256, r - 255, r - 129, r - 128, r - 127, r - 2, r - 1]
    rows = sorted(set([x for x in fixed if 0 <= x < r] + list(rng.integers(0, r, size=n))))
    return np.array(rows)


def _run_full_and_sampled(spec_full, spec_of_rows, laws, seed, row_inputs, rows_total):
    """GPU on the full spec; oracle on spec_of_rows(len(rows)) with row-shaped inputs sliced."""
    import torch
    import paper_2506_10401_b200 as hct
    t = configs.draw_inputs(spec_full, laws, seed)
    g = hct.FusedGraph(spec_full, 0)
    outs = g.run(parity.to_device(spec_full, t))
    torch.cuda.synchronize()
    g.status()
    rows = _sample_rows(rows_total)
    small = {k: (v[rows] if k in row_inputs else v) for k, v in t.items()}
    spec_small = spec_of_rows(len(rows))
    ref = parity.oracle_reference(spec_small, parity.oracle_inputs(spec_small, small))
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
    assert "tcgen05" in g.plan and "CTA pairs" in g.plan
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


def test_config4_full_size_all_images():
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16")
    got, want, g = parity.run_both(spec, laws, 0)
    assert "tcgen05" in g.plan
    assert got[0].shape == (32, 128, 56, 56)
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


def _device_fill(shape, law, dtype, gen):
    import torch
    if law["kind"] == "normal":
        t = torch.randn(shape, device="cuda", generator=gen) * law.get("std", 1.0) + law.get("mean", 0.0)
    elif law["kind"] == "uniform":
        t = torch.rand(shape, device="cuda", generator=gen) * (law["hi"] - law["lo"]) + law["lo"]
    else:
        raise ValueError(law["kind"])
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _full_size_sampled(make, seed):
    """`make(rows=None|m)` -> (spec, laws, meta).  Runs the graph at its drawn row count and compares the sampled rows."""
    import torch
    import paper_2506_10401_b200 as hct
    spec, laws, meta = make(None)
    r_total = meta["rows"]
    rows = _sample_rows(r_total)
    spec_small, laws_small, _ = make(len(rows))
    weights = set(re.findall(r"gemm\(\w+,\s*(\w+)\)", spec))
    small = configs.draw_inputs(spec_small, laws_small, seed)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    idx = torch.from_numpy(rows).cuda()
    ins = []
    for (name, dtype, shape), dev_small in zip(configs.parse_inputs(spec), parity.to_device(spec_small, small)):
        if len(shape) == 2 and shape[0] == r_total and name not in weights and tuple(dev_small.shape) != tuple(shape):
            full = _device_fill(shape, laws[name], dtype, gen)
            full[idx] = dev_small
            ins.append(full)
        else:
            assert tuple(dev_small.shape) == tuple(shape), (name, shape, dev_small.shape)
            ins.append(dev_small)
    g = hct.FusedGraph(spec, 0)
    outs = g.run(ins)
    torch.cuda.synchronize()
    g.status()
    ref = parity.oracle_reference(spec_small, parity.oracle_inputs(spec_small, small))
    worst = 0.0
    for o, (name, _, _) in zip(outs, g.outputs):
        assert o.shape[0] == r_total
        worst = max(worst, parity.f32_violation(parity.to_numpy64(o[idx]), ref[name]))
    assert worst <= 1.0, f"seed {seed}: violated by factor {worst:.3g}\n{g.plan}"
    g.close()


@pytest.mark.parametrize("seed", list(range(200)))
def test_sweep_graph_full_size_sampled_rows(seed):
    _full_size_sampled(lambda m: sweep.get(seed, rows=m), seed)


@pytest.mark.parametrize("seed", list(range(60)))
def test_grown_graph_full_size_sampled_rows(seed):
    _full_size_sampled(lambda m: sweep.get_grown(seed, rows=m), seed)
