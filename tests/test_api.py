"""Host-side behaviour of the C-ABI library: exports, parsing and validation codes, shape
inference against the oracle's independent reader, fusion plans, kernel compilation.  No GPU."""
import ctypes
import os
import re

import pytest

import oracle
import paper_2506_10401_b200 as hct
from paper_2506_10401_b200 import binding
from workloads import configs, sweep

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NONE = hct.HCT_DEVICE_NONE


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "hct.h")).read()
    declared = set(re.findall(r"HCT_API[^;(]*?\b(hct_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    raw = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name
    assert "sm_100a" in hct.hct_version()


def _code(spec):
    with pytest.raises(hct.HctError) as e:
        hct.hct_graph_create(spec, NONE)
    return e.value.code


def test_error_codes():
    assert _code("") == hct.HCT_ERR_PARSE
    assert _code("hct 2\n") == hct.HCT_ERR_PARSE
    assert _code("hct 1\ninput x f64 [4]\n") == hct.HCT_ERR_PARSE
    assert _code("hct 1\ninput x f32 [4,8\nnode y = relu(x)\noutput y\n") == hct.HCT_ERR_PARSE
    assert _code("hct 1\ninput x f32 [4,8]\nnode y relu(x)\noutput y\n") == hct.HCT_ERR_PARSE
    assert _code("hct 1\ninput x f32 [4,8]\nfrob y\n") == hct.HCT_ERR_PARSE
    g = hct.HCT_ERR_GRAPH
    assert _code("hct 1\ninput x f32 [4,8]\nnode y = relu(z)\noutput y\n") == g            # dangling operand
    assert _code("hct 1\ninput x f32 [4,8]\nnode y = add(y, x)\noutput y\n") == g          # cycle
    assert _code("hct 1\ninput x f32 [4,8]\nnode a = relu(b)\nnode b = relu(a)\noutput b\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\ninput v f32 [7]\nnode y = add(x, v)\noutput y\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\ninput w f32 [9,3]\nnode y = gemm(x, w)\noutput y\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\ninput w bf16 [8,3]\nnode y = gemm(x, w)\noutput y\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\nnode y = relu(x)\nnode z = exp(x)\noutput y\n") == g  # z dangles
    assert _code("hct 1\ninput x f32 [4,8]\ninput u f32 [4,8]\nnode y = relu(x)\noutput y\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\nnode y = frobnicate(x)\noutput y\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\nnode y = relu(x)\nnode y = exp(x)\noutput y\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\nnode s = row_sum(x)\nnode y = row_max(s)\noutput y\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\nnode y = relu(x)\n") == g
    assert _code("hct 1\ninput x f32 [4,8]\noutput x\n") == g
    assert _code("hct 1\ninput x f32 [0,8]\nnode y = relu(x)\noutput y\n") == hct.HCT_ERR_UNSUPPORTED
    with pytest.raises(hct.HctError) as e:
        hct.hct_graph_create("hct 1\ninput x f32 [4,8]\nnode y = relu(q)\noutput y\n", NONE)
    assert "line 3" in e.value.message and "'q'" in e.value.message


def test_null_arguments():
    L = hct.lib()
    out = ctypes.c_void_p()
    assert L.hct_graph_create(None, 0, NONE, ctypes.byref(out)) == hct.HCT_ERR_INVALID_ARG
    assert L.hct_graph_create(b"hct 1", 5, NONE, None) == hct.HCT_ERR_INVALID_ARG
    assert L.hct_graph_destroy(None) == hct.HCT_OK
    assert L.hct_graph_run(None, None, 0, None, 0, None, 0, None) == hct.HCT_ERR_INVALID_ARG
    assert L.hct_graph_num_inputs(None) == -1


def test_run_without_device_is_refused():
    spec, _ = configs.get_config("c2_softmax_layernorm_chain", r=8, c=64)
    g = hct.hct_graph_create(spec, NONE)
    with pytest.raises(hct.HctError) as e:
        hct.hct_graph_run(g, [16] * 5, [16])
    assert e.value.code == hct.HCT_ERR_INVALID_ARG
    hct.hct_graph_destroy(g)


def _agree_with_oracle_reader(spec):
    og = oracle.parse(spec)
    g = hct.hct_graph_create(spec, NONE)
    try:
        assert hct.hct_graph_num_inputs(g) == len(og.inputs)
        assert hct.hct_graph_num_outputs(g) == len(og.outputs)
        for i, name in enumerate(og.inputs):
            n, d, s = hct.hct_graph_tensor_info(g, False, i)
            assert (n, s) == (name, tuple(og.nodes[name].shape))
            assert d == (hct.HCT_BF16 if og.nodes[name].dtype == "bf16" else hct.HCT_F32)
        for i, (name, dtype) in enumerate(og.outputs):
            n, d, s = hct.hct_graph_tensor_info(g, True, i)
            assert (n, s) == (name, tuple(og.nodes[name].shape))
            assert d == (hct.HCT_BF16 if dtype == "bf16" else hct.HCT_F32)
        return hct.hct_graph_num_kernels(g), hct.hct_graph_plan_text(g), hct.hct_graph_cost(g), hct.hct_graph_workspace_bytes(g)
    finally:
        hct.hct_graph_destroy(g)


def test_configs_plan_to_one_kernel_each_and_costs():
    k, plan, (b, f), ws = _agree_with_oracle_reader(configs.get_config("c2_softmax_layernorm_chain")[0])
    assert k == 1 and ws == 0 and f == 0 and b == 2 * 8192 * 4096 * 4 + 4 * 4096 * 4
    k, plan, (b, f), ws = _agree_with_oracle_reader(configs.get_config("c1_gemm_bias_relu_f32")[0])
    assert f == 2 * 256 ** 3 and b == 3 * 256 * 256 * 4 + 1024
    k, plan, (b, f), ws = _agree_with_oracle_reader(configs.get_config("c3_gemm_bf16_gelu_residual")[0])
    assert f == 2 * 8192 * 4096 * 4096 and b == (8192 * 4096 * 3 + 4096 * 4096 + 4096) * 2
    k, plan, (b, f), ws = _agree_with_oracle_reader(configs.get_config("c4_conv_bn_relu_bf16")[0])
    assert f == 2 * 32 * 128 * 56 * 56 * 128 * 9 and b == 2 * 32 * 128 * 56 * 56 * 2 + 128 * 128 * 9 * 2 + 2 * 128 * 4


def test_shape_inference_agrees_on_sweep():
    for seed in range(0, 200, 7):
        spec, _, _ = sweep.get(seed, rows=64)
        _agree_with_oracle_reader(spec)


def test_shape_inference_agrees_on_grown_graphs():
    for seed in range(0, 60, 6):
        spec, _, _ = sweep.get_grown(seed, rows=64)
        _agree_with_oracle_reader(spec)


def test_plan_cuts_and_workspace():
    spec = """hct 1
input x f32 [64,256]
input w f32 [256,128]
input b f32 [128]
node a = relu(x)
node s = row_sum(a)
node c = div(a, s)
node m = gemm(c, w)
node d = add(m, b)
node e = row_softmax(d)
output e
output s
"""
    g = hct.hct_graph_create(spec, NONE)
    plan = hct.hct_graph_plan_text(g)
    assert "kernel 0 row [64,256]: a=relu s=row_sum c=div" in plan
    assert "kernel 1 gemm [64,128]: m=gemm d=add" in plan
    assert "kernel 2 row [64,128]: e=row_softmax" in plan
    # c and d cross kernel boundaries through fp32 workspace
    assert hct.hct_graph_workspace_bytes(g) >= (64 * 256 + 64 * 128) * 4
    bytes_, flops = hct.hct_graph_cost(g)
    assert flops == 2 * 64 * 256 * 128
    # inputs + outputs + the operand edge into the gemm (c); d -> softmax is narrower than one accumulator tile
    assert bytes_ == (64 * 256 + 256 * 128 + 128) * 4 + (64 * 128 + 64) * 4 + 8 * 64 * 256
    src = hct.hct_graph_kernel_source(g, 0)
    assert "hct_row_g0" in src and hct.hct_graph_kernel_name(g, 0) == "hct_row_g0"
    hct.hct_graph_destroy(g)


def test_unsupported_broadcast_is_reported_not_emulated():
    spec = "hct 1\ninput x f32 [4,3,8]\ninput v f32 [4,1,8]\nnode y = add(x, v)\noutput y\n"
    assert _code(spec) == hct.HCT_ERR_UNSUPPORTED


def test_row_longer_than_the_limit_is_unsupported():
    assert _code("hct 1\ninput x f32 [2,131076]\nnode y = row_softmax(x)\noutput y\n") == hct.HCT_ERR_UNSUPPORTED


def test_schedule_text_selects_launch_shapes_and_rejects_unknown_knobs():
    B = binding
    spec, _ = configs.get_config("c2_softmax_layernorm_chain", r=64, c=4096)
    a = B.hct_graph_create_scheduled(spec, B.HCT_DEVICE_NONE, None)
    b = B.hct_graph_create_scheduled(spec, B.HCT_DEVICE_NONE, "row_nv=2; row_cta_small=512")
    assert B.hct_graph_schedule(a) == "" and B.hct_graph_schedule(b) == "row_nv=2; row_cta_small=512"
    assert "#define HCT_T 256" in B.hct_graph_kernel_source(a, 0) and "#define HCT_T 512" in B.hct_graph_kernel_source(b, 0)
    for bad in ("no_such_knob=1", "row_nv", "row_nv=four"):
        with pytest.raises(B.HctError) as e:
            B.hct_graph_create_scheduled(spec, B.HCT_DEVICE_NONE, bad)
        assert e.value.code == B.HCT_ERR_INVALID_ARG
    B.hct_graph_destroy(a)
    B.hct_graph_destroy(b)


def test_extents_out_of_range_are_rejected_not_wrapped():
    """An extent that does not fit a 64-bit integer, and shapes whose element count would overflow, are errors of
    the spec (the parser must not wrap them into small numbers and plan a kernel)."""
    import paper_2506_10401_b200 as hct
    for dims in ("[99999999999999999999,4]", "[4294967296,4294967296]", "[1099511627777]", "[2097152,1048576,2]"):
        spec = f"hct 1\ninput x f32 {dims}\nnode y = relu(x)\noutput y\n"
        with pytest.raises(hct.HctError) as e:
            hct.hct_graph_create(spec, hct.HCT_DEVICE_NONE)
        assert e.value.code in (hct.HCT_ERR_PARSE, hct.HCT_ERR_UNSUPPORTED), dims
    spec = "hct 1\ninput x f32 [8,64]\nnode y = dropout(x, p=0.5, seed=99999999999999999999)\noutput y\n"
    with pytest.raises(hct.HctError):
        hct.hct_graph_create(spec, hct.HCT_DEVICE_NONE)


def test_layout_words_on_inputs_and_outputs():
    """`nhwc` on an input or an output is a statement about the caller's buffer: extents stay [N,C,H,W].  Both readers
    accept and reject the same specs; an nhwc output must come out of a convolution kernel."""
    conv = "hct 1\ninput x bf16 [2,16,8,8] nhwc\ninput w bf16 [8,16,3,3]\nnode y = conv2d(x, w, pad=1)\nnode z = relu(y)\n"
    h = hct.hct_graph_create(conv + "output z bf16 nhwc\n", NONE)
    assert binding.hct_graph_input_layout(h, 0) == 1 and binding.hct_graph_input_layout(h, 1) == 0
    assert binding.hct_graph_output_layout(h, 0) == 1 and binding.hct_graph_output_layout(h, 1) == -1
    assert binding.hct_graph_tensor_info(h, True, 0)[2] == (2, 8, 8, 8)
    hct.hct_graph_destroy(h)
    g = oracle.parse(conv + "output z bf16 nhwc\n")
    assert g.output_layouts == {"z": "nhwc"} and g.nodes["z"].shape == (2, 8, 8, 8)
    h = hct.hct_graph_create(conv + "output z bf16 nchw\n", NONE)
    assert binding.hct_graph_output_layout(h, 0) == 0
    hct.hct_graph_destroy(h)
    assert oracle.parse(conv + "output z bf16 nchw\n").output_layouts == {}
    for tail, code in (("output z bf16 nwhc\n", hct.HCT_ERR_PARSE), ("output z bf16 nhwc extra\n", hct.HCT_ERR_PARSE)):
        assert _code(conv + tail) == code
        with pytest.raises(oracle.SpecError):
            oracle.parse(conv + tail)
    flat = "hct 1\ninput x f32 [4,8]\nnode y = relu(x)\noutput y f32 nhwc\n"          # rank 2
    assert _code(flat) == hct.HCT_ERR_UNSUPPORTED
    with pytest.raises(oracle.SpecError):
        oracle.parse(flat)
    # a rank-4 value that no convolution kernel stores: valid spec, not supported by this library
    rows = "hct 1\ninput x f32 [2,3,4,8]\nnode y = relu(x)\noutput y f32 nhwc\n"
    oracle.parse(rows)
    assert _code(rows) == hct.HCT_ERR_UNSUPPORTED
