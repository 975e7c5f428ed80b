"""The fp32 parity criterion itself, checked on the CPU.

The criterion must be (i) the strict relative 1e-5 wherever nothing cancels, (ii) the condition
number of the sum for a cancelling row sum, (iii) satisfiable: the oracle's own definitions
evaluated in float32 by numpy (a legitimate single-precision implementation that shares nothing
with the CUDA kernels) must pass it on the sweep graphs, and (iv) sharp: a planted relative error
of 3e-5 on one element of a well-conditioned output must fail it."""
import math

import numpy as np
import pytest

import oracle
from tests import errbound, parity
from workloads import configs, sweep

N_ = {"kind": "normal", "mean": 0.0, "std": 1.0}


def _ref(spec, laws, seed=0):
    t = configs.draw_inputs(spec, laws, seed)
    ins = parity.oracle_inputs(spec, t)
    return parity.oracle_reference(spec, ins), ins


def test_chains_without_cancellation_are_judged_at_strict_relative_tolerance():
    spec = """hct 1
input x f32 [40,300]
node a = exp(x)
node s = sigmoid(a)
node q = sqrt(s)
node r = rsqrt(q)
node c = reciprocal(r)
node d = square(c)
node e = relu(d)
node f = mul(e, a)
node p = row_softmax(s)
node m = row_max(p)
node n = row_min(f)
node t = row_sum(f)
node u = row_mean(s)
output e
output p
output m
output n
output t
output u
"""
    ref, _ = _ref(spec, {"x": N_})
    for name, r in ref.items():
        bound, strict = parity.f32_bound(r)
        np.testing.assert_array_equal(bound, np.maximum(strict, parity.FLOOR), err_msg=name)


def test_cancelling_row_sum_is_scaled_by_the_sum_of_magnitudes():
    spec = "hct 1\ninput x f32 [30,4096]\nnode s = row_sum(x)\nnode m = row_mean(x)\noutput s\noutput m\n"
    ref, ins = _ref(spec, {"x": N_})
    cond = np.abs(ins["x"]).sum(axis=1, keepdims=True)
    np.testing.assert_allclose(ref["s"].err, (math.log2(4096) + 1) * 2.0 ** -24 * cond, rtol=1e-12)
    bound, strict = parity.f32_bound(ref["s"])
    # the allowance is a small multiple of u * sum|x| (below 1e-5 * sum|x|), and it is what decides these rows
    assert np.all(bound <= 1e-5 * cond) and np.all(bound >= strict)
    assert np.mean(bound > strict) > 0.5
    # same-sign terms: nothing cancels and the criterion is strict again
    ref, _ = _ref(spec, {"x": {"kind": "uniform", "lo": 0.5, "hi": 2.0}})
    bound, strict = parity.f32_bound(ref["s"])
    np.testing.assert_array_equal(bound, strict)


def test_full_width_bound_is_never_looser_than_the_row_scale_rule():
    spec, laws = configs.get_config("c2_softmax_layernorm_chain", r=32, c=1024)
    ref, _ = _ref(spec, laws)
    r = ref["t4"]
    bound, _ = parity.f32_bound(r)
    assert np.all(bound <= 1e-5 * np.maximum(np.abs(np.asarray(r)), parity.row_scale(r)) + 1e-300)
    # x - mean cancels in a layer normalisation: most elements get an allowance above the strict bound,
    # and it stays far below the row-scale rule on average
    assert np.median(bound / (1e-5 * parity.row_scale(r))) < 0.2


def _float32_run(spec, ins):
    g = oracle.parse(spec)
    seq = lambda a, b: np.matmul(a.astype(np.float32), b.astype(np.float32))
    val = oracle.run_nodes(g, {k: v.astype(np.float32) for k, v in ins.items()}, dtype=np.float32, gemm_fn=seq)
    return {name: val[name].astype(np.float64) for name, _ in g.outputs}


@pytest.mark.parametrize("seed", list(range(0, 200, 4)))
def test_numpy_float32_evaluation_passes_the_criterion(seed):
    spec, laws, _ = sweep.get(seed, rows=24)
    ref, ins = _ref(spec, laws, seed)
    got = _float32_run(spec, ins)
    for name in ref:
        assert parity.f32_violation(got[name], ref[name]) <= 1.0, (seed, name)


def test_planted_relative_error_fails_where_nothing_cancels():
    spec = "hct 1\ninput x f32 [16,256]\nnode a = sigmoid(x)\nnode p = row_softmax(a)\noutput p\n"
    ref, ins = _ref(spec, {"x": N_})
    got = np.array(ref["p"])
    assert parity.f32_violation(got, ref["p"]) == 0.0
    j = np.unravel_index(np.argmin(got), got.shape)       # the smallest element of the output
    got[j] *= 1.0 + 3e-5
    assert parity.f32_violation(got, ref["p"]) > 1.0
