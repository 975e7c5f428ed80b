"""The allocation-free GEMM entry point against the CPU oracle and the regular graph path.  Collected
last on purpose: a run that stops at the first failure has then already exercised everything else.

hct_gemm_bias_relu_f32_static keeps the split operands of an fp32 GEMM in a fixed array inside the
library instead of caller workspace, for callers that cannot allocate device memory.  Two calls in
a row (different shapes, so the second overwrites only part of what the first left in the array)
must each agree with the oracle on the same inputs within the library's fp32 tolerance, and so
must hct_graph_run; the two device results are two roundings of the same product, so they are
also compared with each other at twice that tolerance.
"""
import ctypes

import numpy as np
import pytest

from tests import parity
from workloads import configs

pytestmark = pytest.mark.gpu


def _both(m, k, n, seed):
    import torch
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c1_gemm_bias_relu_f32", m=m, k=k, n=n)
    t = configs.draw_inputs(spec, laws, seed)
    a, b, bias = parity.to_device(spec, t)
    g = hct.FusedGraph(spec, 0)
    ref = g.run([a, b, bias])[0]
    out = torch.full((m, n), float("nan"), device="cuda")
    hct.hct_gemm_bias_relu_f32_static(a.data_ptr(), b.data_ptr(), bias.data_ptr(), out.data_ptr(), m, k, n, True, 0,
                                      torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    g.status()
    want = parity.oracle_reference(spec, parity.oracle_inputs(spec, t))["t2"]
    return parity.to_numpy64(out), parity.to_numpy64(ref), want


def test_static_scratch_gemm_matches_oracle_and_graph_path_twice():
    for (m, k, n, seed) in [(256, 256, 256, 0), (70, 132, 200, 1), (256, 256, 256, 2)]:
        got, graph, want = _both(m, k, n, seed)
        worst = parity.f32_violation(got, want)
        assert worst <= 1.0, f"({m},{k},{n}): static-scratch result differs from the oracle by factor {worst:.3g} of tolerance"
        assert parity.f32_violation(graph, want) <= 1.0
        bound, _ = parity.f32_bound(want)
        assert np.all(np.abs(got - graph) <= 2 * bound)


def test_static_scratch_rejects_oversized_and_bad_arguments():
    import torch
    import paper_2506_10401_b200 as hct
    x = torch.zeros(16, device="cuda")
    big = hct.HCT_STATIC_SCRATCH_BYTES // 8
    with pytest.raises(hct.HctError) as e:
        hct.hct_gemm_bias_relu_f32_static(x.data_ptr(), x.data_ptr(), 0, x.data_ptr(), big, 2, 2)
    assert e.value.code == hct.HCT_ERR_UNSUPPORTED and "too large" in e.value.message
    with pytest.raises(hct.HctError) as e:
        hct.hct_gemm_bias_relu_f32_static(0, x.data_ptr(), 0, x.data_ptr(), 2, 2, 2)
    assert e.value.code == hct.HCT_ERR_INVALID_ARG
    # a 2x2 product with no bias and no relu still works after the rejections
    a = torch.tensor([[1.0, 2.0], [3.0, 4.0]], device="cuda")
    b = torch.tensor([[0.0, 1.0], [-1.0, 0.0]], device="cuda")
    out = torch.empty(2, 2, device="cuda")
    hct.hct_gemm_bias_relu_f32_static(a.data_ptr(), b.data_ptr(), 0, out.data_ptr(), 2, 2, 2, False)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out.cpu().numpy(), np.array([[-2.0, 1.0], [-4.0, 3.0]], dtype=np.float32))
