"""Parity of the CUDA library against the CPU oracle on identical seeded inputs.  Needs a B200."""
import numpy as np
import pytest

from tests import parity
from workloads import configs, sweep

pytestmark = pytest.mark.gpu

N_ = {"kind": "normal", "mean": 0.0, "std": 1.0}
POS_ = {"kind": "uniform", "lo": 0.5, "hi": 2.0}


def check_f32(spec, laws, seed=0):
    got, want, g = parity.run_both(spec, laws, seed)
    worst = max(parity.f32_violation(a, b) for a, b in zip(got, want))
    assert worst <= 1.0, f"fp32 parity violated by factor {worst:.3g}\n{g.plan}"
    return g


def check_bf16(spec, laws, seed=0):
    got, want, g = parity.run_both(spec, laws, seed)
    worst = max(parity.bf16_violation(a, b) for a, b in zip(got, want))
    assert worst <= 1.0, f"bf16 parity violated by factor {worst:.3g}\n{g.plan}"
    return g


# ------------------------------------------------------------------ memory-bound chains

@pytest.mark.parametrize("std,c", [(1e-3, 4096), (30.0, 4096), (1.0, 2560), (1e-3, 8192), (8.0, 16384)])
def test_layernorm_of_softmax_takes_variance_from_the_softmax_sums(std, c):
    """Near-uniform rows (variance far below 1/C^2) and nearly one-hot rows are the two ends of the
    cancellation in mean(p^2) - 1/C^2; both must stay inside the fp32 tolerance."""
    spec, laws = configs.get_config("c2_softmax_layernorm_chain", r=64, c=c)
    laws = dict(laws)
    laws["x"] = {"kind": "normal", "mean": 0.0, "std": std}
    g = check_f32(spec, laws)
    assert g.num_kernels == 1


@pytest.mark.parametrize("r,c", [(300, 4096), (37, 1000), (5, 1023), (64, 130), (1, 4096), (129, 256), (33, 8192), (7, 20000), (3, 65536), (2, 131072)])
def test_softmax_layernorm_chain_shapes(r, c):
    spec, laws = configs.get_config("c2_softmax_layernorm_chain", r=r, c=c)
    g = check_f32(spec, laws)
    assert g.num_kernels == 1


@pytest.mark.parametrize("schedule", [None, "row_no_packed=1"])
@pytest.mark.parametrize("body,cols", [
    # three sigmoids and a softmax on few bytes: the reciprocals run as Newton steps on the multiply-add pipe
    ("node a = sigmoid(x)\nnode b = sigmoid(a)\nnode c = add(b, v)\nnode d = sigmoid(c)\nnode e = row_softmax(d)\noutput e\noutput d\n", 4096),
    # products folded into sums in every operand order, and a softmax whose scaling is NOT left to the layer norm (two readers)
    ("node a = mul(x, v)\nnode b = sub(a, x)\nnode m = mul(b, v)\nnode c = sub(x, m)\nnode p = row_softmax(c)\n"
     "node l = row_layernorm(p, v, v, eps=1e-5)\nnode o = add(l, p)\noutput o\n", 4096),
    # ragged rows: pairs for the elementwise part, one-value reductions
    ("node a = mul(x, v)\nnode b = add(a, v)\nnode g = gelu_tanh(b)\nnode p = row_softmax(g)\nnode l = row_layernorm(p, v, v, eps=1e-5)\noutput l\n", 1000),
    ("node a = sigmoid(x)\nnode b = mul(a, 3.0)\nnode c = add(b, v)\nnode s = row_sum(c)\noutput c\noutput s\n", 4094),
])
def test_packed_pairs_and_one_value_arithmetic_agree_with_the_oracle(body, cols, schedule):
    spec = f"hct 1\ninput x f32 [70,{cols}]\ninput v f32 [{cols}]\n" + body
    got, want, g = parity.run_both(spec, {"x": {"kind": "normal", "mean": 0.0, "std": 3.0}, "v": N_}, schedule=schedule)
    for a, b in zip(got, want):
        assert parity.f32_violation(a, b) <= 1.0, g.plan


def test_sigmoid_far_out_in_both_tails():
    """Arguments up to +-200: beyond -87.3 the exponential's argument is kept at 126 and the result is below the
    smallest normal number, as the exact value is; +200 gives exactly one."""
    spec = "hct 1\ninput x f32 [8,4096]\nnode a = sigmoid(x)\nnode b = sigmoid(a)\nnode c = sigmoid(b)\nnode d = sigmoid(c)\nnode e = sigmoid(d)\noutput a\noutput e\n"
    got, want, g = parity.run_both(spec, {"x": {"kind": "uniform", "lo": -200.0, "hi": 200.0}})
    assert "hct_sigmoid2(hct_pk(" in g.kernel_source(0)   # the variant with Newton steps
    for a, b in zip(got, want):
        assert parity.f32_violation(a, b) <= 1.0, g.plan


def test_two_column_rows():
    spec = "hct 1\ninput x f32 [3,2]\nnode y = row_softmax(x)\nnode s = row_sum(y)\noutput y\noutput s\n"
    check_f32(spec, {"x": N_})


@pytest.mark.parametrize("op", ["relu", "gelu_tanh", "gelu_erf", "sigmoid", "exp", "tanh", "sqrt", "sin", "cos", "neg", "abs", "log", "rsqrt",
                                "square", "reciprocal"])
def test_unary(op):
    spec = f"hct 1\ninput x f32 [67,200]\nnode y = {op}(x)\noutput y\n"
    check_f32(spec, {"x": POS_ if op in ("sqrt", "log", "rsqrt", "reciprocal") else N_})


@pytest.mark.parametrize("op", ["add", "sub", "mul", "div", "max", "min"])
def test_binary_broadcast_kinds(op):
    spec = f"""hct 1
input x f32 [45,132]
input full f32 [45,132]
input rowv f32 [132]
input colv f32 [45,1]
input one f32 [1]
node a = {op}(x, full)
node b = {op}(a, rowv)
node c = {op}(colv, b)
node d = {op}(c, 1.5)
node e = {op}(0.75, d)
node f = {op}(e, one)
output f
output b
"""
    check_f32(spec, {"x": POS_, "full": POS_, "rowv": POS_, "colv": POS_, "one": POS_})


def test_row_reductions_and_column_values():
    spec = """hct 1
input x f32 [70,777]
node s = row_sum(x)
node m = row_mean(x)
node mx = row_max(x)
node c = sub(x, m)
node n = div(c, mx)
node t = tanh(s)
node y = mul(n, t)
output y
output s
output m
output mx
"""
    check_f32(spec, {"x": POS_})


def test_bf16_input_and_output_rows():
    spec = "hct 1\ninput x bf16 [50,264]\ninput b bf16 [264]\nnode t = add(x, b)\nnode y = row_softmax(t)\noutput y bf16\n"
    got, want, g = parity.run_both(spec, {"x": N_, "b": N_})
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


def test_channel_broadcast_rank4():
    spec = "hct 1\ninput x f32 [3,5,6,20]\ninput s f32 [5,1,1]\ninput t f32 [1,5,1,1]\nnode a = mul(x, s)\nnode y = add(a, t)\noutput y\n"
    check_f32(spec, {"x": N_, "s": N_, "t": N_})


# ------------------------------------------------------------------ contractions

def test_config1_gemm_bias_relu_full_size():
    spec, laws = configs.get_config("c1_gemm_bias_relu_f32")
    check_f32(spec, laws)


@pytest.mark.parametrize("m,k,n", [(1, 1, 1), (5, 7, 3), (130, 260, 72), (300, 1000, 520), (64, 4096, 128), (128, 16384, 128), (2, 8, 4100)])
def test_gemm_f32_shapes(m, k, n):
    spec, laws = configs.get_config("c1_gemm_bias_relu_f32", m=m, k=k, n=n)
    check_f32(spec, laws)


@pytest.mark.parametrize("m,k,n", [(300, 1000, 520), (257, 4096, 136), (130, 264, 1000), (1024, 260, 300), (64, 36, 257)])
def test_gemm_f32_wide_tiles(m, k, n):
    """128 x 256 tiles of the fp32 (three TF32 products) kernel, whose running sums are shared by eight epilogue warps,
    forced onto small and ragged shapes (by rule they are taken when narrower tiles need more than one round)."""
    import torch
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c1_gemm_bias_relu_f32", m=m, k=k, n=n)
    t = configs.draw_inputs(spec, laws, 0)
    g = hct.FusedGraph(spec, 0, schedule="gemm_bn=256;gemm_pair=2")
    assert "128x256x32" in g.plan
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    ref = parity.oracle_reference(spec, parity.oracle_inputs(spec, t))["t2"]
    assert parity.f32_violation(parity.to_numpy64(out), ref) <= 1.0
    il = {"kind": "int", "lo": -8, "hi": 8}
    t = configs.draw_inputs(spec, {"a": il, "b": il, "bias": il}, 1)
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    np.testing.assert_array_equal(parity.to_numpy64(out), parity.oracle_reference(spec, parity.oracle_inputs(spec, t))["t2"])


@pytest.mark.parametrize("m,k,n", [(300, 1000, 520), (1024, 1024, 1024), (130, 4096, 136), (257, 1028, 264), (70, 16384, 72)])
def test_gemm_f32_contraction_split_over_idle_sms(m, k, n):
    """Few tiles and a deep contraction: the K extent is cut into parts that meet in an accumulation tile in scratch
    (cleared by the pre-pass on every run).  The chain within the fp32 tolerance, twice in a row on one workspace,
    and bit for bit on integer inputs (exact in any order of addition); the same shapes without the split."""
    spec, laws = configs.get_config("c1_gemm_bias_relu_f32", m=m, k=k, n=n)
    got, want, g = parity.run_both(spec, laws, runs=2)
    assert "contraction split" in g.plan
    assert parity.f32_violation(got[0], want[0]) <= 1.0
    il = {"kind": "int", "lo": -8, "hi": 8}
    for schedule in (None, "gemm_no_ksplit=1"):
        got, want, g = parity.run_both(spec, {"a": il, "b": il, "bias": il}, schedule=schedule, runs=2)
        assert ("contraction split" in g.plan) == (schedule is None)
        np.testing.assert_array_equal(got[0], want[0])


def test_gemm_f32_integer_inputs_are_exact():
    spec, _ = configs.get_config("c1_gemm_bias_relu_f32", m=96, k=160, n=136)
    il = {"kind": "int", "lo": -8, "hi": 8}
    got, want, _ = parity.run_both(spec, {"a": il, "b": il, "bias": il})
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("m,k,n", [(300, 264, 520), (128, 64, 256), (1, 8, 8), (257, 4096, 136), (2048, 512, 1024), (130, 16384, 72)])
def test_gemm_bf16_chain_shapes(m, k, n):
    spec, laws = configs.get_config("c3_gemm_bf16_gelu_residual", m=m, k=k, n=n)
    check_bf16(spec, laws)


@pytest.mark.parametrize("m,k,n", [(300, 264, 520), (257, 4096, 136), (1, 8, 8), (512, 64, 512), (130, 1000, 264), (1000, 320, 776)])
def test_gemm_bf16_on_cta_pairs(m, k, n):
    """The CTA-pair kernel (256 x 256 tiles, chosen by rule only for large problems) forced onto small and ragged shapes."""
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c3_gemm_bf16_gelu_residual", m=m, k=k, n=n)
    t = configs.draw_inputs(spec, laws, 0)
    g = hct.FusedGraph(spec, 0, schedule="gemm_pair=1")
    assert "CTA pairs" in g.plan
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    ref = oracle.run(spec, parity.oracle_inputs(spec, t))["t3"]
    assert parity.bf16_violation(parity.to_numpy64(out), ref) <= 1.0
    # integer-valued operands: every partial sum is exact, so the product must match bit for bit
    spec = f"hct 1\ninput x bf16 [{m},{k}]\ninput w bf16 [{k},{n}]\nnode y = gemm(x, w)\noutput y f32\n"
    il = {"kind": "int", "lo": -8, "hi": 8}
    t = configs.draw_inputs(spec, {"x": il, "w": il}, 1)
    g = hct.FusedGraph(spec, 0, schedule="gemm_pair=1")
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    np.testing.assert_array_equal(parity.to_numpy64(out), oracle.run(spec, parity.oracle_inputs(spec, t))["y"])


@pytest.mark.parametrize("m,k,n", [(300, 1000, 520), (257, 4096, 136), (1, 4, 4), (512, 64, 256), (130, 16384, 72), (1024, 260, 1000), (64, 36, 100)])
def test_gemm_f32_split_inside_the_kernel(m, k, n):
    """One launch, no scratch: the kernel splits fp32 operands into TF32 head and tail itself (forced here; by rule for small problems)."""
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c1_gemm_bias_relu_f32", m=m, k=k, n=n)
    t = configs.draw_inputs(spec, laws, 0)
    g = hct.FusedGraph(spec, 0, schedule="gemm_insplit=1")
    assert "split in the kernel" in g.plan and g.num_kernels == 1 and g.workspace_bytes == 0
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    ref = parity.oracle_reference(spec, parity.oracle_inputs(spec, t))["t2"]
    assert parity.f32_violation(parity.to_numpy64(out), ref) <= 1.0
    il = {"kind": "int", "lo": -8, "hi": 8}
    t = configs.draw_inputs(spec, {"a": il, "b": il, "bias": il}, 1)
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    np.testing.assert_array_equal(parity.to_numpy64(out), oracle.run(spec, parity.oracle_inputs(spec, t))["t2"])


@pytest.mark.parametrize("m,k,n", [(300, 1000, 520), (257, 4096, 136), (5, 8, 3), (512, 64, 256), (130, 16384, 72), (1024, 260, 1000)])
def test_gemm_f32_on_cta_pairs(m, k, n):
    """The fp32 (three TF32 products) kernel on CTA pairs, forced onto small and ragged shapes."""
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c1_gemm_bias_relu_f32", m=m, k=k, n=n)
    t = configs.draw_inputs(spec, laws, 0)
    g = hct.FusedGraph(spec, 0, schedule="gemm_pair=1")
    assert "CTA pairs" in g.plan
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    ref = parity.oracle_reference(spec, parity.oracle_inputs(spec, t))["t2"]
    assert parity.f32_violation(parity.to_numpy64(out), ref) <= 1.0
    il = {"kind": "int", "lo": -8, "hi": 8}
    t = configs.draw_inputs(spec, {"a": il, "b": il, "bias": il}, 1)
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    np.testing.assert_array_equal(parity.to_numpy64(out), oracle.run(spec, parity.oracle_inputs(spec, t))["t2"])


def test_gemm_bf16_integer_inputs_are_exact():
    spec = "hct 1\ninput x bf16 [200,320]\ninput w bf16 [320,264]\nnode y = gemm(x, w)\noutput y f32\n"
    il = {"kind": "int", "lo": -8, "hi": 8}
    got, want, _ = parity.run_both(spec, {"x": il, "w": il})
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("kw", [
    dict(n=2, c=128, h=14, w=14, k=128),
    dict(n=1, c=128, h=56, w=56, k=128),
    dict(n=3, c=64, h=9, w=11, k=32),
    dict(n=2, c=3, h=8, w=8, k=5, ksize=1, pad=0),
    dict(n=1, c=8, h=12, w=10, k=4, stride=2, pad=1),
    dict(n=1, c=4, h=7, w=7, k=4, ksize=3, pad=0),
    # rows of a multiple of 8 pixels: the kernel reads NCHW itself
    dict(n=2, c=64, h=20, w=24, k=96),
    dict(n=1, c=72, h=17, w=40, k=130, ksize=5, pad=2),
    dict(n=3, c=128, h=6, w=64, k=64, ksize=1, pad=0),
    dict(n=1, c=16, h=33, w=56, k=128, ksize=3, pad=0),
    dict(n=2, c=8, h=5, w=120, k=8, ksize=3, pad=2),
])
def test_conv_chain_shapes(kw):
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16", **kw)
    check_bf16(spec, laws)


@pytest.mark.parametrize("kw", [
    dict(n=2, c=128, h=56, w=56, k=128),                       # tiles start in the middle of rows; 13 tiles per image, the last one short
    dict(n=1, c=72, h=17, w=48, k=130, ksize=5, pad=2),        # four dropped positions per row, two blocks of output channels
    dict(n=3, c=128, h=6, w=64, k=64, ksize=1, pad=0),         # no dropped positions at all
    dict(n=1, c=16, h=33, w=56, k=128, ksize=3, pad=0),        # no padding: the pitch is the image width
    dict(n=2, c=8, h=5, w=88, k=8, ksize=3, pad=1),            # rows longer than two chunks
    dict(n=1, c=64, h=9, w=48, k=32, ksize=3, pad=2),          # padding wider than half the filter: output rows longer than input rows
])
def test_conv_flat_tiles(kw):
    """Tiles of 256 consecutive positions (chosen by rule only when they save a K loop), forced onto other shapes:
    the chain within the bf16 tolerance, and the bare convolution bit for bit on integer-valued inputs."""
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16", **kw)
    ks, pad = kw.get("ksize", 3), kw.get("pad", 1)
    schedule = "conv_flat=1" + (";conv_no_pointwise=1" if ks == 1 else "")
    got, want, g = parity.run_both(spec, laws, schedule=schedule)
    assert "flat tiles" in g.plan
    assert parity.bf16_violation(got[0], want[0]) <= 1.0
    spec = (f"hct 1\ninput x bf16 [{kw['n']},{kw['c']},{kw['h']},{kw['w']}]\ninput w bf16 [{kw['k']},{kw['c']},{ks},{ks}]\n"
            f"node y = conv2d(x, w, stride=1, pad={pad})\nnode z = cast_bf16(y)\noutput z bf16\n")
    il = {"kind": "int", "lo": -2, "hi": 2}
    got, want, g = parity.run_both(spec, {"x": il, "w": il}, schedule=schedule)
    assert "flat tiles" in g.plan
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("kw,out", [
    (dict(n=11, c=128, h=56, w=56, k=128), "bf16"),                    # 154 tiles: 6 left over, 6 parts per row
    (dict(n=11, c=64, h=56, w=56, k=128), "f32"),                      # one channel block: 3 parts; fp32 result without TMA stores
    (dict(n=15, c=192, h=40, w=56, k=128), "bf16"),                    # three channel blocks: 9 parts
    (dict(n=19, c=64, h=30, w=56, k=256), "bf16"),                     # two filter blocks, last tile of an image two rows high
    (dict(n=15, c=72, h=17, w=48, k=130, ksize=5, pad=2), "bf16"),     # 5x5 filter, ragged channel and filter blocks: 10 parts
])
def test_conv_last_round_split_by_part_of_the_contraction(kw, out):
    """Schedule conv_ksplit=1: with a few tiles more than a multiple of the grid, the left-over rows are cut by (channel
    block, filter row) part; partial sums meet in scratch and the last part to arrive finishes the row.  Shapes chosen for a grid of 148
    CTAs; the chain within the bf16 tolerance and the bare convolution bit for bit on integer inputs, twice in a row
    on one workspace (every run clears the arrival counters), and the same under the default schedule."""
    import torch
    if torch.cuda.get_device_properties(0).multi_processor_count != 148:
        pytest.skip("tile counts chosen for 148 SMs")
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16", **kw)
    got, want, g = parity.run_both(spec, laws, schedule="conv_ksplit=1")
    assert "NCHW read directly" in g.plan
    assert parity.bf16_violation(got[0], want[0]) <= 1.0
    ks, pad = kw.get("ksize", 3), kw.get("pad", 1)
    tail = "node z = cast_bf16(y)\noutput z bf16\n" if out == "bf16" else "output y f32\n"
    spec = (f"hct 1\ninput x bf16 [{kw['n']},{kw['c']},{kw['h']},{kw['w']}]\ninput w bf16 [{kw['k']},{kw['c']},{ks},{ks}]\n"
            f"node y = conv2d(x, w, stride=1, pad={pad})\n" + tail)
    il = {"kind": "int", "lo": -2, "hi": 2}
    for schedule in ("conv_ksplit=1", None):
        got, want, g = parity.run_both(spec, {"x": il, "w": il}, schedule=schedule, runs=2 if schedule else 1)
        np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("shape,wshape,attrs", [
    ((2, 64, 28, 30), (96, 64, 3, 3), "stride=2, pad=1"),             # strided pixel boxes straight from the caller's buffer
    ((1, 128, 56, 56), (256, 128, 1, 1), "stride=2, pad=0"),
    ((2, 64, 20, 24), (96, 64, 3, 3), "stride=1, pad=1"),             # stride 1: pixels shared by the taps of a filter row
    ((1, 72, 17, 40), (130, 72, 5, 5), "stride=1, pad=2"),
    ((3, 8, 9, 11), (32, 8, 3, 3), "stride=1, pad=1"),                # small image: one box per tap
    ((1, 8, 6, 300), (8, 8, 3, 3), "stride=2, pad=1"),                # stride-phase view of the caller's buffer
    ((1, 8, 16, 32), (16, 8, 3, 3), "stride=4, pad=1, dilation=3"),
])
def test_conv_channels_last_input_is_read_in_place(shape, wshape, attrs):
    """An input declared nhwc: same values as the NCHW graph, channels-last in memory; the convolution reads the
    caller's buffer through its tensor maps and the only pre-pass left is the one over the weights."""
    dims = lambda t: "[" + ",".join(str(v) for v in t) + "]"
    spec = f"hct 1\ninput x bf16 {dims(shape)} nhwc\ninput w bf16 {dims(wshape)}\nnode y = conv2d(x, w, {attrs})\noutput y f32\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il})
    assert "channels-last input read in place" in g.plan and "weight pre-pass" in g.plan and "NHWC activations" not in g.plan
    assert g.workspace_bytes <= 256 + 2 * int(np.prod(wshape))
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("body", [
    "input x bf16 [2,64,14,16]\ninput w bf16 [96,64,3,3]\nnode y = conv2d(x, w, pad=1)\noutput y bf16 nhwc\n",               # one box per tap
    "input x bf16 [2,64,14,16] nhwc\ninput w bf16 [96,64,3,3]\nnode y = conv2d(x, w, stride=2, pad=1)\noutput y f32 nhwc\n",   # channels-last in and out
    "input x bf16 [2,32,56,56]\ninput w bf16 [72,32,1,1]\nnode y = conv2d(x, w)\noutput y bf16 nhwc\n",                        # per-image GEMM
    "input x bf16 [2,128,20,56]\ninput w bf16 [130,128,3,3]\nnode y = conv2d(x, w, pad=1)\noutput y f32 nhwc\n",               # NCHW read directly
    "input x bf16 [1,72,17,40] nhwc\ninput w bf16 [40,72,5,5]\nnode y = conv2d(x, w, pad=2)\noutput y bf16 nhwc\n",             # pixels shared by a filter row
    "input x bf16 [2,16,12,24]\ninput w bf16 [16,1,3,3]\nnode y = conv2d(x, w, pad=1, groups=16)\noutput y bf16 nhwc\n",        # depthwise, 8 columns per thread
    "input x bf16 [1,6,9,7]\ninput w bf16 [6,1,3,3]\nnode y = conv2d(x, w, pad=1, groups=6)\noutput y f32 nhwc\n",              # depthwise, one column per thread
    "input x f32 [2,6,8,8]\ninput w f32 [4,6,3,3]\nnode y = conv2d(x, w, pad=1)\noutput y f32 nhwc\n",                          # fp32-FMA kernel
    "input x bf16 [2,64,14,16]\ninput w bf16 [64,32,3,3]\nnode y = conv2d(x, w, pad=1, groups=2)\noutput y bf16 nhwc\n",        # grouped
])
def test_conv_channels_last_output(body):
    """An output declared nhwc: same values as the NCHW graph, written channels-last into the caller's buffer."""
    import torch
    # a bf16 output is rounded: state the rounding as a node, so that the oracle's value is the rounded one
    spec = "hct 1\n" + body.replace("output y bf16 nhwc", "node z = cast_bf16(y)\noutput z bf16 nhwc")
    il = {"kind": "int", "lo": -4, "hi": 4}
    t = configs.draw_inputs(spec, {"x": il, "w": il}, 0)
    ref = list(parity.oracle_reference(spec, parity.oracle_inputs(spec, t)).values())[0]
    g = hct_graph(spec)
    assert g.output_nhwc == [True]
    out = g.run(parity.to_device(spec, t))[0]
    torch.cuda.synchronize()
    g.status()
    assert out.is_contiguous(memory_format=torch.channels_last) and tuple(out.shape) == ref.shape
    np.testing.assert_array_equal(parity.to_numpy64(out), ref)
    # the buffer itself, read as [N,H,W,C]
    raw = torch.as_strided(out, (out.shape[0], out.shape[2], out.shape[3], out.shape[1]),
                           (out.shape[1] * out.shape[2] * out.shape[3], out.shape[3] * out.shape[1], out.shape[1], 1))
    np.testing.assert_array_equal(parity.to_numpy64(raw), np.transpose(np.asarray(ref), (0, 2, 3, 1)))


def test_conv_channels_last_between_two_graphs():
    """A channels-last pipeline across graphs: the first graph's nhwc output is the second graph's nhwc input, with no
    layout pass over the activations in either; compared with the oracle's run of the two convolutions as one graph."""
    import torch
    one = ("hct 1\ninput x bf16 [2,64,28,28] nhwc\ninput w1 bf16 [128,64,3,3]\ninput s f32 [128,1,1]\nnode a = conv2d(x, w1, stride=2, pad=1)\n"
           "node b = mul(a, s)\nnode c = relu(b)\noutput c bf16 nhwc\n")
    two = "hct 1\ninput c bf16 [2,128,14,14] nhwc\ninput w2 bf16 [64,128,3,3]\nnode y = conv2d(c, w2, pad=1)\noutput y f32 nhwc\n"
    both = ("hct 1\ninput x bf16 [2,64,28,28]\ninput w1 bf16 [128,64,3,3]\ninput s f32 [128,1,1]\ninput w2 bf16 [64,128,3,3]\n"
            "node a = conv2d(x, w1, stride=2, pad=1)\nnode b = mul(a, s)\nnode c0 = relu(b)\nnode c = cast_bf16(c0)\nnode y = conv2d(c, w2, pad=1)\noutput y f32\n")
    il = {"kind": "int", "lo": -2, "hi": 2}
    t = configs.draw_inputs(both, {"x": il, "w1": il, "w2": il, "s": {"kind": "int", "lo": 1, "hi": 2}}, 0)
    ref = parity.oracle_reference(both, parity.oracle_inputs(both, t))["y"]
    dev = dict(zip(["x", "w1", "s", "w2"], parity.to_device(both, t)))
    g1, g2 = hct_graph(one), hct_graph(two)
    assert "NHWC activations" not in g1.plan and "NHWC activations" not in g2.plan
    c = g1.run([dev["x"].contiguous(memory_format=torch.channels_last), dev["w1"], dev["s"]])[0]
    y = g2.run([c, dev["w2"]])[0]
    torch.cuda.synchronize()
    g1.status(); g2.status()
    np.testing.assert_array_equal(parity.to_numpy64(y), ref)


def hct_graph(spec, schedule=None):
    import paper_2506_10401_b200 as hct
    return hct.FusedGraph(spec, 0, schedule=schedule)


def test_conv_channels_last_chain():
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16", n=2, c=64, h=56, w=56, k=128, stride=2, pad=1, nhwc=True)
    check_bf16(spec, laws)


def test_conv_f32_integer_inputs_are_exact():
    spec = "hct 1\ninput x f32 [2,16,10,12]\ninput w f32 [8,16,3,3]\nnode y = conv2d(x, w, stride=1, pad=1)\noutput y\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, _ = parity.run_both(spec, {"x": il, "w": il})
    np.testing.assert_array_equal(got[0], want[0])


def test_conv_bf16_nchw_direct_integer_inputs_are_exact():
    spec = "hct 1\ninput x bf16 [2,80,13,48]\ninput w bf16 [40,80,3,3]\nnode y = conv2d(x, w, stride=1, pad=1)\noutput y f32\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il})
    assert "NCHW read directly" in g.plan
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("shape,wshape,attrs", [
    ((2, 64, 28, 30), (96, 64, 3, 3), "stride=2, pad=1"),
    ((1, 128, 56, 56), (256, 128, 1, 1), "stride=2, pad=0"),          # downsampling 1x1
    ((2, 16, 23, 19), (40, 16, 3, 3), "stride=3, pad=1"),             # extents not divisible by the stride: strided boxes
    ((2, 16, 24, 18), (40, 16, 3, 3), "stride=3, pad=1"),
    ((1, 8, 16, 32), (16, 8, 3, 3), "stride=4, pad=1, dilation=3"),
    ((3, 24, 12, 16), (20, 24, 5, 5), "stride=2, pad=4"),             # padding beyond half the filter
    ((1, 8, 40, 72), (16, 8, 5, 5), "stride=8, pad=2"),
    ((1, 72, 21, 26), (130, 72, 3, 3), "stride=1, pad=2, dilation=2"),
    ((2, 8, 25, 31), (8, 8, 3, 2), "stride=2, pad=3, dilation=3"),
    ((1, 8, 40, 70), (16, 8, 5, 5), "stride=8, pad=2"),
    ((1, 8, 6, 300), (8, 8, 3, 3), "stride=2, pad=1"),
    ((1, 8, 6, 301), (8, 8, 3, 3), "stride=2, pad=1"),                # too wide for one strided box: fp32-FMA kernel
])
@pytest.mark.parametrize("schedule", [None, "conv_phase=1"])
def test_conv_bf16_stride_and_dilation_integer_inputs_are_exact(shape, wshape, attrs, schedule):
    dims = lambda t: "[" + ",".join(str(v) for v in t) + "]"
    spec = f"hct 1\ninput x bf16 {dims(shape)}\ninput w bf16 {dims(wshape)}\nnode y = conv2d(x, w, {attrs})\noutput y f32\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il}, schedule=schedule)
    assert ("pixel boxes" in g.plan) == (shape[3] != 301)
    stride = int(attrs[7])
    divisible = stride > 1 and shape[2] % stride == 0 and shape[3] % stride == 0
    assert ("stride-phase view" in g.plan) == (divisible and (schedule is not None or shape[3] == 300))
    np.testing.assert_array_equal(got[0], want[0])


def test_conv_strided_chain_and_f32_dilation():
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16", n=2, c=64, h=56, w=56, k=128, stride=2, pad=1)
    check_bf16(spec, laws)
    spec = "hct 1\ninput x f32 [2,6,11,12]\ninput w f32 [5,6,3,3]\nnode y = conv2d(x, w, stride=2, pad=2, dilation=2)\noutput y\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, _ = parity.run_both(spec, {"x": il, "w": il})
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("dtype,shape,wshape,attrs", [
    ("bf16", (2, 32, 28, 28), (32, 1, 3, 3), "pad=1, groups=32"),
    ("bf16", (1, 24, 57, 41), (24, 1, 3, 3), "stride=2, pad=1, groups=24"),
    ("f32", (1, 4, 9, 9), (8, 1, 3, 3), "stride=2, pad=1, groups=4"),                # two filters per channel
    ("f32", (2, 5, 13, 11), (5, 1, 5, 5), "pad=2, groups=5"),
    ("bf16", (1, 6, 17, 19), (6, 1, 3, 3), "pad=2, dilation=2, groups=6"),
    ("f32", (1, 3, 2, 70), (3, 1, 3, 3), "pad=1, groups=3"),                         # fewer output rows than a thread's block
    ("f32", (1, 2, 30, 9), (2, 1, 7, 7), "stride=3, pad=3, groups=2"),
    # rows of whole 16-byte vectors at stride 1: blocks of 8 columns per thread
    ("bf16", (2, 16, 12, 24), (16, 1, 3, 3), "pad=1, groups=16"),
    ("f32", (1, 3, 7, 16), (6, 1, 5, 5), "pad=2, groups=3"),
    ("f32", (1, 4, 5, 40), (4, 1, 1, 1), "groups=4"),
    ("bf16", (1, 4, 9, 16), (4, 1, 5, 3), "pad=1, groups=4"),                        # 7 output rows: ragged last block
    ("bf16", (3, 8, 1, 8), (8, 1, 3, 3), "pad=1, groups=8"),                         # a single output row
    ("bf16", (2, 6, 8, 7), (4, 3, 3, 2), "pad=1, dilation=2, groups=2"),             # grouped, not depthwise
    ("f32", (1, 8, 6, 6), (12, 2, 1, 1), "groups=4"),
])
def test_conv_groups_integer_inputs_are_exact(dtype, shape, wshape, attrs):
    dims = lambda t: "[" + ",".join(str(v) for v in t) + "]"
    spec = f"hct 1\ninput x {dtype} {dims(shape)}\ninput w {dtype} {dims(wshape)}\nnode y = conv2d(x, w, {attrs})\noutput y f32\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il})
    assert ("depthwise" in g.plan) == (wshape[1] == 1)
    assert ("8 columns" in g.plan) == (wshape[1] == 1 and shape[3] % 8 == 0)
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("shape,ko", [
    ((2, 32, 56, 56), 192),      # expansion of an inverted-residual block: two channel blocks, 13 pixel blocks, the last one short
    ((3, 192, 14, 28), 32),      # projection: three blocks of input channels, a quarter of the MMA rows used
    ((1, 72, 6, 12), 130),       # 72 pixels, channels not a multiple of 64, two filters in the second channel block
    ((2, 8, 2, 4), 8),           # one 16-byte row per channel
    ((1, 200, 33, 24), 40),      # 792 pixels: three full blocks and 24 pixels
    ((5, 64, 16, 16), 256),      # whole tiles only
])
def test_conv_pointwise_is_a_per_image_gemm(shape, ko):
    """1x1 convolution, stride 1, no padding, on NCHW data: weights and pixels are read where they lie.  Bare result
    bit for bit on integer-valued inputs through both store paths (fp32: the generated epilogue's own stores;
    bf16: shared memory and TMA stores), then a chain with per-channel operands and a residual within the bf16 tolerance."""
    n, c, h, w = shape
    il = {"kind": "int", "lo": -4, "hi": 4}
    head = f"hct 1\ninput x bf16 [{n},{c},{h},{w}]\ninput w bf16 [{ko},{c},1,1]\n"
    got, want, g = parity.run_both(head + "node y = conv2d(x, w)\noutput y f32\n", {"x": il, "w": il})
    assert "per-image GEMM" in g.plan and g.num_kernels == 1 and g.workspace_bytes <= 256
    np.testing.assert_array_equal(got[0], want[0])
    got, want, g = parity.run_both(head + "node y = conv2d(x, w)\nnode z = cast_bf16(y)\noutput z bf16\n", {"x": il, "w": il})
    assert "per-image GEMM" in g.plan and g.num_kernels == 1
    np.testing.assert_array_equal(got[0], want[0])
    spec = (head + f"input s f32 [{ko},1,1]\ninput b f32 [{ko},1,1]\ninput r bf16 [{n},{ko},{h},{w}]\n"
            "node y = conv2d(x, w)\nnode a = mul(y, s)\nnode c = add(a, b)\nnode d = relu(c)\nnode e = add(d, r)\noutput e bf16\n")
    nrm = {"kind": "normal", "mean": 0.0, "std": 1.0}
    got, want, g = parity.run_both(spec, {"x": nrm, "w": {"kind": "normal", "mean": 0.0, "std": c ** -0.5}, "s": {"kind": "uniform", "lo": 0.5, "hi": 1.5},
                                          "b": nrm, "r": nrm})
    assert "per-image GEMM" in g.plan
    assert parity.bf16_violation(got[0], want[0]) <= 1.0
    # the general schedules stay available and agree
    got2, _, g2 = parity.run_both(spec, {"x": nrm, "w": {"kind": "normal", "mean": 0.0, "std": c ** -0.5}, "s": {"kind": "uniform", "lo": 0.5, "hi": 1.5},
                                         "b": nrm, "r": nrm}, schedule="conv_no_pointwise=1")
    assert "per-image GEMM" not in g2.plan
    assert parity.bf16_violation(got2[0], want[0]) <= 1.0


@pytest.mark.parametrize("shape,wshape,attrs,nhwc,window", [
    ((2, 64, 14, 16), (64, 32, 3, 3), "pad=1, groups=2", False, 64),                 # one block of filters spans both groups
    ((1, 256, 12, 12), (256, 64, 3, 3), "pad=1, groups=4", False, 128),              # two blocks of filters, two groups each
    ((1, 72, 9, 20), (192, 24, 3, 3), "pad=1, groups=3", False, 64),                 # windows start at channels 0 and 48; both run past their groups
    ((1, 64, 16, 16), (96, 16, 3, 3), "stride=2, pad=1, groups=4", False, 64),       # strided pixel boxes
    ((2, 256, 10, 10), (512, 128, 1, 1), "groups=2", False, 128),                    # a block of filters lies inside one group: nothing wasted
    ((1, 128, 9, 20), (128, 4, 3, 3), "pad=1, groups=32", False, 128),               # four channels per group
    ((1, 128, 20, 56), (128, 32, 3, 3), "pad=1, groups=4", False, 128),              # pixels shared by the taps of a filter row
    ((2, 64, 14, 16), (64, 32, 3, 3), "pad=1, groups=2", True, 64),                  # channels-last input read in place
    ((1, 128, 20, 56), (256, 32, 3, 3), "pad=1, groups=4", True, 64),
])
def test_conv_grouped_on_tensor_cores(shape, wshape, attrs, nhwc, window):
    """1 < groups < channels: each block of 128 filters contracts the dense window of input channels its groups span,
    against a weight copy that is zero outside every filter's own group.  Bit for bit on integer-valued inputs."""
    dims = lambda t: "[" + ",".join(str(v) for v in t) + "]"
    spec = (f"hct 1\ninput x bf16 {dims(shape)}{' nhwc' if nhwc else ''}\ninput w bf16 {dims(wshape)}\n"
            f"node y = conv2d(x, w, {attrs})\noutput y f32\n")
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il})
    assert "tcgen05" in g.plan and f"dense windows of {window} input channels" in g.plan
    np.testing.assert_array_equal(got[0], want[0])


def test_conv_grouped_window_off_a_16_byte_boundary_takes_the_fma_kernel():
    spec = "hct 1\ninput x bf16 [1,24,8,8]\ninput w bf16 [256,12,3,3]\nnode y = conv2d(x, w, pad=1, groups=2)\noutput y f32\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il})
    assert "fp32-FMA" in g.plan
    np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("dtype,shape,wshape,attrs", [
    ("bf16", (2, 16, 12, 24), (16, 1, 3, 3), "pad=1, groups=16"),
    ("f32", (1, 3, 7, 16), (6, 1, 5, 5), "pad=2, groups=3"),                         # two filters per channel: a pair shares its input plane
    ("f32", (1, 4, 5, 40), (4, 1, 1, 1), "groups=4"),
    ("bf16", (1, 4, 9, 16), (4, 1, 5, 3), "pad=1, groups=4"),
    ("bf16", (3, 8, 1, 8), (8, 1, 3, 3), "pad=1, groups=8"),
    ("bf16", (2, 32, 56, 56), (32, 1, 3, 3), "pad=1, groups=32"),
])
def test_depthwise_two_filters_per_thread(dtype, shape, wshape, attrs):
    """The opt-in schedule with packed multiply-adds (filters k and k+1 in the two halves): same results bit for bit."""
    dims = lambda t: "[" + ",".join(str(v) for v in t) + "]"
    spec = f"hct 1\ninput x {dtype} {dims(shape)}\ninput w {dtype} {dims(wshape)}\nnode y = conv2d(x, w, {attrs})\noutput y f32\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il}, schedule="dw_pair=1")
    assert "two filters per thread" in g.plan
    np.testing.assert_array_equal(got[0], want[0])
    spec, laws = configs.get_config("dwconv_bn_relu", n=2, c=48, h=28, w=24)
    got, want, g = parity.run_both(spec, laws, schedule="dw_pair=1")
    assert "two filters per thread" in g.plan
    got1, _, _ = parity.run_both(spec, laws)
    np.testing.assert_array_equal(got[0], got1[0])      # each half is an ordinary fused multiply-add
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


@pytest.mark.parametrize("kw", [dict(n=2, c=48, h=28, w=28), dict(n=1, c=16, h=15, w=21, stride=2), dict(n=2, c=192, h=56, w=56)])
def test_depthwise_chain(kw):
    spec, laws = configs.get_config("dwconv_bn_relu", **kw)
    check_bf16(spec, laws)


@pytest.mark.parametrize("kw", [dict(n=2, c=32, h=28, w=24), dict(n=1, c=16, h=14, w=14, expand=4), dict(n=2, c=32, h=56, w=56)])
def test_inverted_residual_block(kw):
    spec, laws = configs.get_config("mbconv_block", **kw)
    got, want, g = parity.run_both(spec, laws)
    assert g.plan.count("tcgen05") == 2 and g.plan.count("depthwise") == 1
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


@pytest.mark.parametrize("kw", [dict(n=1, c=8, h=8, w=8, expand=2, blocks=3, c_out=16), dict(n=2, c=32, h=28, w=24, blocks=3, c_out=64),
                                dict(n=2, c=16, h=56, w=56, expand=6, blocks=2, c_out=24)])
def test_mobilenet_stage(kw):
    """Several inverted-residual blocks and a stride-2 transition as ONE graph: nine convolution kernels, every
    activation between them kept as bf16 on the device."""
    spec, laws = configs.get_config("mobilenet_stage", **kw)
    got, want, g = parity.run_both(spec, laws)
    assert g.plan.count("depthwise") == kw["blocks"] and g.num_kernels >= 3 * kw["blocks"]
    outside, worst = parity.bf16_deep_chain_check(got[0], want[0])
    assert outside <= 1e-3 and worst <= 1.0, (outside, worst)


@pytest.mark.parametrize("kw", [dict(n=1, c=32, h=6, w=8, width=16, groups=2), dict(n=2, c=256, h=28, w=28), dict(n=1, c=64, h=14, w=14, width=64, groups=4)])
def test_resnext_block(kw):
    """A bottleneck whose 3x3 convolution is grouped: all three convolutions on tensor cores."""
    spec, laws = configs.get_config("resnext_block", **kw)
    got, want, g = parity.run_both(spec, laws)
    assert g.plan.count("tcgen05") == 3 and "dense windows" in g.plan
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


# ------------------------------------------------------------------ stacked contractions through bf16 intermediates

@pytest.mark.parametrize("kw", [dict(n=2, c=64, h=20, w=24, k=64), dict(n=1, c=128, h=56, w=56, k=128), dict(n=2, c=16, h=9, w=11, k=32)])
def test_conv_block_keeps_bf16_activations_on_the_device(kw):
    spec, laws = configs.get_config("conv_block", **kw)
    got, want, g = parity.run_both(spec, laws)
    assert g.plan.count("tcgen05") == 2       # both convolutions on tensor cores
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


def test_gemm_chain_through_cast_bf16():
    spec = """hct 1
input x  bf16 [300,264]
input w1 bf16 [264,520]
input b1 bf16 [520]
input w2 bf16 [520,136]
node h0 = gemm(x, w1)
node h1 = add(h0, b1)
node h2 = gelu_tanh(h1)
node h3 = cast_bf16(h2)
node y  = gemm(h3, w2)
output y f32
output h3 bf16
"""
    n = {"kind": "normal", "mean": 0.0, "std": 1.0}
    got, want, g = parity.run_both(spec, {"x": n, "w1": {"kind": "normal", "mean": 0.0, "std": 0.06}, "b1": n,
                                          "w2": {"kind": "normal", "mean": 0.0, "std": 0.04}})
    assert g.plan.count("tcgen05") == 2 and g.num_kernels == 2
    assert parity.bf16_violation(got[0], want[0]) <= 1.0
    assert parity.bf16_violation(got[1], want[1]) <= 1.0


# ------------------------------------------------------------------ layout transform

@pytest.mark.parametrize("r,c", [(37, 1000), (300, 4096), (5, 1023), (1, 7), (64, 64), (129, 65), (2048, 2048)])
def test_transpose_is_exact_and_fuses_its_consumers(r, c):
    spec = f"hct 1\ninput x f32 [{r},{c}]\ninput b f32 [{r}]\ninput y bf16 [{r},{c}]\nnode t = transpose(x)\nnode u = add(t, b)\nnode v = relu(u)\n" \
           f"node w = transpose(y)\noutput t\noutput v\noutput w bf16\n"
    n = {"kind": "normal", "mean": 0.0, "std": 1.0}
    got, want, g = parity.run_both(spec, {"x": n, "b": n, "y": n})
    np.testing.assert_array_equal(got[0], want[0])     # pure data movement
    np.testing.assert_array_equal(got[2], want[2])     # bf16 in, bf16 out: exact too
    assert parity.f32_violation(got[1], want[1]) <= 1.0
    assert g.num_kernels == 2 and "transpose" in g.plan


@pytest.mark.parametrize("shape,axes", [((2, 6, 5, 7), "0231"), ((2, 6, 5, 7), "0312"), ((3, 70, 9, 66), "0231"), ((2, 3, 4, 5), "3210"),
                                        ((4, 5, 6), "102"), ((4, 5, 6), "210"), ((130, 67), "10"), ((2, 3, 65, 130), "1032"),
                                        ((2, 6, 5, 7), "1023"), ((5, 3, 2, 64), "2103"), ((1, 128, 28, 28), "0231")])
def test_permute_is_exact_and_fuses_its_consumers(shape, axes):
    """Pure data movement (bit for bit, fp32 and bf16), with elementwise consumers applied at the store."""
    dims = "[" + ",".join(str(v) for v in shape) + "]"
    last = shape[int(axes[-1])]
    spec = (f"hct 1\ninput x f32 {dims}\ninput y bf16 {dims}\ninput b f32 [{last}]\nnode p = permute(x, axes={axes})\nnode q = add(p, b)\n"
            f"node r = relu(q)\nnode s = permute(y, axes={axes})\noutput p\noutput r\noutput s bf16\n")
    got, want, g = parity.run_both(spec, {"x": N_, "y": N_, "b": N_})
    assert g.num_kernels == 2 and g.plan.count("permute") >= 2
    np.testing.assert_array_equal(got[0], want[0])
    np.testing.assert_array_equal(got[2], want[2])
    assert parity.f32_violation(got[1], want[1]) <= 1.0


def test_permute_to_channels_last_and_back_around_a_row_kernel():
    spec = """hct 1
input x f32 [2,16,6,8]
input g f32 [16]
input b f32 [16]
node a = permute(x, axes=0231)
node f = reshape(a, rows=96, cols=16)
node n = row_layernorm(f, g, b, eps=1e-5)
output n
"""
    check_f32(spec, {"x": N_, "g": POS_, "b": N_})


def test_transpose_between_other_kernels():
    spec = """hct 1
input x f32 [96,256]
input w f32 [96,128]
input g f32 [128]
input b f32 [128]
node a = gelu_tanh(x)
node t = transpose(a)
node m = gemm(t, w)
node n = row_layernorm(m, g, b, eps=1e-5)
node o = transpose(n)
output o
"""
    n = {"kind": "normal", "mean": 0.0, "std": 1.0}
    got, want, g = parity.run_both(spec, {"x": n, "w": {"kind": "normal", "mean": 0.0, "std": 0.1}, "g": n, "b": n})
    assert got[0].shape == (128, 256)
    assert parity.f32_violation(got[0], want[0]) <= 1.0


# ------------------------------------------------------------------ arg reductions (indices are exact)

@pytest.mark.parametrize("r,c", [(37, 1000), (300, 4096), (5, 1023), (64, 130), (3, 65536), (129, 24)])
def test_row_argmax_argmin_min(r, c):
    # taken on the inputs themselves (and on exact maps of them), so both sides see the same values
    spec = f"hct 1\ninput x f32 [{r},{c}]\nnode a = row_argmax(x)\nnode n = neg(x)\nnode b = row_argmin(n)\nnode q = relu(x)\n" \
           f"node c = row_argmin(q)\nnode d = row_min(x)\nnode e = row_argmin(x)\noutput a\noutput b\noutput c\noutput d\noutput e\n"
    got, want, g = parity.run_both(spec, {"x": {"kind": "normal", "mean": 0.0, "std": 1.0}})
    for a, b in zip(got, want):
        np.testing.assert_array_equal(a, b)      # relu makes many equal zeros: the first column must win


def test_row_argmax_after_inexact_chain_points_at_a_maximum():
    # after rounding arithmetic the winner may differ between fp32 and fp64: what is checked is that the
    # reported column holds a value within the fp32 tolerance of the row maximum
    import oracle
    spec = "hct 1\ninput x f32 [200,3000]\ninput w f32 [3000]\nnode t = mul(x, w)\nnode u = gelu_tanh(t)\nnode a = row_argmax(u)\noutput a\noutput u\n"
    n = {"kind": "normal", "mean": 0.0, "std": 1.0}
    got, want, g = parity.run_both(spec, {"x": n, "w": n})
    idx = got[0][:, 0].astype(np.int64)
    assert np.all((idx >= 0) & (idx < 3000))
    u = want[1]
    top = u.max(axis=1)
    picked = u[np.arange(200), idx]
    assert np.all(top - picked <= 1e-5 * np.abs(u).max(axis=1))


# ------------------------------------------------------------------ dropout (counter-based mask)

def _mask_is_exact(got, want):
    """The mask is integer work: dropped elements are exactly zero on both sides, in the same places."""
    np.testing.assert_array_equal(got == 0.0, want == 0.0)


@pytest.mark.parametrize("r,c,p,seed", [(37, 1000, 0.3, 5), (300, 4096, 0.5, 123456789), (5, 1023, 0.0, 1), (3, 65536, 0.9, (1 << 40) + 7),
                                        (64, 130, 0.25, 0)])
def test_dropout_in_row_chain(r, c, p, seed):
    spec = f"hct 1\ninput x f32 [{r},{c}]\ninput b f32 [{c}]\nnode a = add(x, b)\nnode d = dropout(a, p={p}, seed={seed})\n" \
           f"node s = row_sum(d)\nnode e = dropout(s, p=0.5, seed={seed + 1})\noutput d\noutput e\n"
    n = {"kind": "normal", "mean": 0.5, "std": 1.0}
    got, want, g = parity.run_both(spec, {"x": n, "b": n})
    _mask_is_exact(got[0], want[0])
    _mask_is_exact(got[1], want[1])
    assert max(parity.f32_violation(a, b) for a, b in zip(got, want)) <= 1.0
    assert g.num_kernels == 1


def test_dropout_in_gemm_and_conv_epilogues():
    spec = "hct 1\ninput x bf16 [300,264]\ninput w bf16 [264,520]\nnode t = gemm(x, w)\nnode d = dropout(t, p=0.4, seed=99)\noutput d f32\n"
    got, want, g = parity.run_both(spec, {"x": {"kind": "normal", "mean": 0.0, "std": 1.0}, "w": {"kind": "normal", "mean": 0.0, "std": 0.06}})
    assert "tcgen05" in g.plan and g.num_kernels == 1
    _mask_is_exact(got[0], want[0])
    assert parity.bf16_violation(got[0], want[0]) <= 1.0
    spec = "hct 1\ninput x bf16 [2,64,20,24]\ninput w bf16 [96,64,3,3]\nnode t = conv2d(x, w, stride=1, pad=1)\nnode d = dropout(t, p=0.3, seed=7)\noutput d bf16\n"
    got, want, g = parity.run_both(spec, {"x": {"kind": "normal", "mean": 0.0, "std": 1.0}, "w": {"kind": "normal", "mean": 0.0, "std": 0.04}})
    assert "tcgen05" in g.plan
    _mask_is_exact(got[0], want[0])
    assert parity.bf16_violation(got[0], want[0]) <= 1.0
    spec = "hct 1\ninput x f32 [1,8,12,10]\ninput w f32 [4,8,3,3]\nnode t = conv2d(x, w, stride=2, pad=1)\nnode d = dropout(t, p=0.3, seed=7)\noutput d\n"
    il = {"kind": "int", "lo": -4, "hi": 4}
    got, want, g = parity.run_both(spec, {"x": il, "w": il})
    _mask_is_exact(got[0], want[0])
    assert parity.f32_violation(got[0], want[0]) <= 1.0


@pytest.mark.parametrize("m,k,n", [(200, 320, 264), (1024, 512, 1024)])
def test_case_study_chain_matmul_dropout_mean_softmax(m, k, n):
    spec, laws = configs.get_config("matmul_dropout_mean_softmax", m=m, k=k, n=n)
    got, want, g = parity.run_both(spec, laws)
    np.testing.assert_array_equal(got[0], np.ones((m, 1)))      # softmax of one value per row
    np.testing.assert_array_equal(want[0], np.ones((m, 1)))
    assert parity.bf16_violation(got[1], want[1]) <= 1.0
    assert parity.f32_violation(got[1], want[1], tol=2e-3) <= 1.0  # mean of bf16-input products: far inside the bf16 class


# ------------------------------------------------------------------ measure-and-pick over schedules

def test_autotune_keeps_results_and_reports_its_choice():
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c2_softmax_layernorm_chain", r=2048, c=4096)
    t = configs.draw_inputs(spec, laws, 0)
    ins = parity.to_device(spec, t)
    g = hct.FusedGraph.autotuned(spec, ins, max_trials=6)
    outs = g.run(ins)
    torch.cuda.synchronize()
    g.status()
    ref = parity.oracle_reference(spec, parity.oracle_inputs(spec, t))["t4"]
    assert parity.f32_violation(parity.to_numpy64(outs[0]), ref) <= 1.0
    # the chosen schedule can be replayed through the plain entry point and gives the same kernels
    again = hct.FusedGraph(spec, 0, schedule=g.schedule)
    assert again.kernel_source(0) == g.kernel_source(0)
    # a convolution graph: the candidates include the other convolution schedules
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16", n=2, h=24, w=24)
    t = configs.draw_inputs(spec, laws, 0)
    ins = parity.to_device(spec, t)
    g = hct.FusedGraph.autotuned(spec, ins, max_trials=4)
    outs = g.run(ins)
    torch.cuda.synchronize()
    g.status()
    ref = oracle.run(spec, parity.oracle_inputs(spec, t))["t3"]
    assert parity.bf16_violation(parity.to_numpy64(outs[0]), ref) <= 1.0


# ------------------------------------------------------------------ multi-kernel graphs

def test_gemm_between_row_kernels():
    spec = """hct 1
input x f32 [96,256]
input w f32 [256,384]
input b f32 [384]
node a = relu(x)
node s = row_sum(a)
node c = div(a, s)
node m = gemm(c, w)
node d = add(m, b)
node e = row_softmax(d)
output e
output s
"""
    g = check_f32(spec, {"x": POS_, "w": N_, "b": N_})
    assert g.num_kernels >= 3


@pytest.mark.parametrize("seed", list(range(200)))
def test_sweep_graphs_reduced_rows(seed):
    """Same random graphs as the sweep, 96 rows each so that the oracle stays fast."""
    spec, laws, _ = sweep.get(seed, rows=96)
    check_f32(spec, laws, seed)


def _rejected_draws():
    return [(e["seed"], a) for e in sweep.entries() for a in range(e["attempt"])]


def _numpy_float32(spec, ins):
    """The oracle's own definitions evaluated in float32 by numpy: a plain single-precision implementation."""
    import oracle
    g = oracle.parse(spec)
    mm = lambda a, b: np.matmul(a.astype(np.float32), b.astype(np.float32))
    with np.errstate(all="ignore"):
        val = oracle.run_nodes(g, {k: v.astype(np.float32) for k, v in ins.items()}, dtype=np.float32, gemm_fn=mm)
    return [val[n].astype(np.float64) for n, _ in g.outputs]


@pytest.mark.parametrize("seed,attempt", _rejected_draws())
def test_sweep_draws_the_conditioning_filter_redrew(seed, attempt):
    """The draws the sweep's conditioning filter replaced (not part of the 200 benchmark graphs).  Many of them
    defeat every float32 evaluation (an exponential of an exponential overflows, or errors grow beyond first
    order), so the yardstick is a plain float32 evaluation of the oracle's definitions by numpy: where that
    stays finite the library must stay finite, and where it sits inside half of the error bound the library
    must meet the bound like on any benchmark graph."""
    from workloads import random_dag
    spec, laws, _ = random_dag.make_dag(seed, attempt, rows=96)
    t = configs.draw_inputs(spec, laws, seed)
    ins = parity.oracle_inputs(spec, t)
    ref = parity.oracle_reference(spec, ins)
    if not all(np.all(np.isfinite(r)) and np.abs(np.asarray(r)).max() < 1e30 for r in ref.values()):
        pytest.skip("the exact values overflow float32: nothing to compare")
    plain = _numpy_float32(spec, ins)
    got, want, g = parity.run_both(spec, laws, seed)
    for a, b, c in zip(got, want, plain):
        if np.all(np.isfinite(c)):
            assert np.all(np.isfinite(a)), "the library overflows where a plain float32 evaluation does not"
            if parity.f32_violation(c, b) <= 0.5:
                worst = parity.f32_violation(a, b)
                assert worst <= 1.0, f"violated by factor {worst:.3g}\n{g.plan}"


# ------------------------------------------------------------------ reshape

@pytest.mark.parametrize("dtype,shape,rows,cols", [("f32", (6, 20), 8, 15), ("bf16", (2, 3, 4, 5), 2, 60), ("f32", (1000,), 8, 125),
                                                    ("bf16", (37, 129), 129, 37), ("f32", (4, 8, 16, 16), 32, 256)])
def test_reshape_moves_values_exactly_and_fuses_consumers(dtype, shape, rows, cols):
    dims = "[" + ",".join(str(v) for v in shape) + "]"
    spec = (f"hct 1\ninput x {dtype} {dims}\ninput b f32 [{cols}]\ninput s f32 [{rows},1]\nnode f = reshape(x, rows={rows}, cols={cols})\n"
            "node u = add(f, b)\nnode v = mul(u, s)\noutput f\noutput v\n")
    got, want, g = parity.run_both(spec, {"x": N_, "b": N_, "s": N_})
    assert g.num_kernels == 1
    np.testing.assert_array_equal(got[0], want[0])
    assert parity.f32_violation(got[1], want[1]) <= 1.0


def test_conv_flatten_gemm_head():
    """conv -> bias -> ReLU -> bf16 -> flatten -> fully connected layer: the flattened activations stay bf16 and feed the tensor-core GEMM."""
    spec = """hct 1
input x  bf16 [64,32,8,8]
input w  bf16 [32,32,3,3]
input b  f32 [32,1,1]
input fc bf16 [2048,256]
input fb f32 [256]
node c0 = conv2d(x, w, pad=1)
node c1 = add(c0, b)
node c2 = relu(c1)
node c3 = cast_bf16(c2)
node f  = reshape(c3, rows=64, cols=2048)
node y0 = gemm(f, fc)
node y  = add(y0, fb)
output y
"""
    wl = {"kind": "normal", "mean": 0.0, "std": 0.06}
    got, want, g = parity.run_both(spec, {"x": N_, "w": wl, "b": N_, "fc": {"kind": "normal", "mean": 0.0, "std": 0.02}, "fb": N_})
    assert "hct_reshape" in g.plan and g.plan.count("tcgen05") == 2
    assert parity.bf16_violation(got[0], want[0]) <= 1.0


# ------------------------------------------------------------------ logic-intensive operators: row sort and top-k

@pytest.mark.parametrize("rows,cols", [(5, 1), (7, 2), (33, 5), (64, 100), (40, 1024), (9, 3000), (6, 4096), (3, 8192)])
@pytest.mark.parametrize("descending", [0, 1])
def test_row_sort_moves_values_exactly(rows, cols, descending):
    spec = f"hct 1\ninput x f32 [{rows},{cols}]\nnode s = row_sort(x, descending={descending})\noutput s\n"
    for law in (N_, {"kind": "int", "lo": -6, "hi": 6}):        # distinct values, and many equal ones
        got, want, g = parity.run_both(spec, {"x": law})
        assert "bitonic" in g.plan
        np.testing.assert_array_equal(got[0], want[0])


@pytest.mark.parametrize("cols,k", [(7, 1), (100, 8), (1000, 1000), (4096, 50), (300, 299)])
def test_row_topk_with_fused_consumers(cols, k):
    spec = (f"hct 1\ninput x bf16 [37,{cols}]\ninput b f32 [{k}]\nnode t = row_topk(x, k={k})\nnode u = add(t, b)\n"
            "node v = relu(u)\noutput t\noutput v\n")
    got, want, g = parity.run_both(spec, {"x": N_, "b": N_})
    assert g.num_kernels == 1
    np.testing.assert_array_equal(got[0], want[0])               # the selected values are inputs, moved unchanged
    assert parity.f32_violation(got[1], want[1]) <= 1.0


@pytest.mark.parametrize("rows,cols,k", [(3, 2, 1), (16, 64, 64), (40, 777, 5), (9, 8192, 256), (21, 4096, 33), (12, 1000, 128)])
@pytest.mark.parametrize("law", ["normal", "ties"])
def test_row_topk_radix_selection_moves_values_exactly(rows, cols, k, law):
    spec = f"hct 1\ninput x f32 [{rows},{cols}]\nnode t = row_topk(x, k={k})\noutput t\n"
    got, want, g = parity.run_both(spec, {"x": N_ if law == "normal" else {"kind": "int", "lo": -3, "hi": 3}})
    assert "radix selection" in g.plan
    np.testing.assert_array_equal(got[0], want[0])
    got2, _, g2 = parity.run_both(spec, {"x": N_ if law == "normal" else {"kind": "int", "lo": -3, "hi": 3}}, schedule="topk_no_select=1")
    assert "bitonic network over" in g2.plan and "radix" not in g2.plan
    np.testing.assert_array_equal(got2[0], want[0])


@pytest.mark.parametrize("rows,cols,k", [(5, 1, 1), (7, 2, 2), (33, 5, 3), (64, 100, 100), (40, 1024, 50), (9, 3000, 7), (6, 4096, 4096), (3, 8192, 256)])
@pytest.mark.parametrize("law", ["normal", "ties"])
def test_row_argsort_and_topk_indices_are_exact(rows, cols, k, law):
    """Columns of the ordered values: index work, compared bit for bit; with many equal values (and both zeros) the
    smaller column must come first in both directions."""
    spec = (f"hct 1\ninput x f32 [{rows},{cols}]\ninput y bf16 [{rows},{cols}]\nnode a = row_argsort(x)\nnode d = row_argsort(y, descending=1)\n"
            f"node t = row_topk_indices(x, k={k})\nnode u = add(t, 0.5)\noutput a\noutput d\noutput t\noutput u\n")
    lw = N_ if law == "normal" else {"kind": "int", "lo": -2, "hi": 2}
    got, want, g = parity.run_both(spec, {"x": lw, "y": lw})
    assert g.plan.count("64-bit (value, column) keys") == 3
    for a, b in zip(got, want):
        np.testing.assert_array_equal(a, b)


def test_row_argsort_treats_both_zeros_as_equal():
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    x = np.array([[0.0, -0.0, 1.0, -0.0, 0.0, -1.0, 0.0, -0.0]] * 3, dtype=np.float32)
    for desc in (0, 1):
        spec = f"hct 1\ninput x f32 [3,8]\nnode a = row_argsort(x, descending={desc})\noutput a\n"
        g = hct.FusedGraph(spec, 0)
        got = g.run([torch.from_numpy(x).cuda()])[0].cpu().numpy().astype(np.float64)
        g.status()
        np.testing.assert_array_equal(got, oracle.run(spec, {"x": x.astype(np.float64)})["a"])


def test_row_topk_when_one_thread_holds_every_large_value():
    """Large values 256 columns apart all belong to one thread of the top-k kernel, so the bound taken from the
    per-thread maxima admits most of the row and the kernel has to fall back to the radix selection."""
    import torch
    import oracle
    import paper_2506_10401_b200 as hct
    rng = np.random.default_rng(5)
    x = rng.normal(size=(6, 4096)).astype(np.float32)
    x[:, ::256] += 100.0
    x[3, :] = np.sort(x[3, :])[::-1]            # one row already in descending order
    for k in (8, 16, 64):
        spec = f"hct 1\ninput x f32 [6,4096]\nnode t = row_topk(x, k={k})\noutput t\n"
        g = hct.FusedGraph(spec, 0)
        got = g.run([torch.from_numpy(x).cuda()])[0].cpu().numpy()
        g.status()
        want = oracle.run(spec, {"x": x.astype(np.float64)})["t"]
        np.testing.assert_array_equal(got.astype(np.float64), want)


@pytest.mark.parametrize("kw", [dict(r=70, c=4096), dict(r=33, c=1000), dict(r=5, c=8192), dict(r=9, c=300)])
def test_sort_config_small(kw):
    """Sort with fused consumers; 512 to 16384 slots take the register kernel, shorter rows the shared-memory one."""
    spec, laws = configs.get_config("sort_bias_relu", **kw)
    check_f32(spec, laws)


def test_topk_config_small():
    spec, laws = configs.get_config("topk_bias_relu", r=96, c=2048, k=32)
    g = check_f32(spec, laws)
    assert g.num_kernels == 1


def test_sort_inside_a_chain():
    spec = """hct 1
input x f32 [50,777]
input w f32 [16,40]
node a = gelu_tanh(x)
node s = row_sort(a)
node p = row_softmax(s)
node t = row_topk(p, k=16)
node y = gemm(t, w)
output y
output s
"""
    g = check_f32(spec, {"x": N_, "w": N_})
    assert g.num_kernels >= 4


@pytest.mark.parametrize("mean,std", [(100.0, 30.0), (-5000.0, 3.0), (0.0, 3e9), (2.5e10, 1e10), (15.9, 0.2)])
@pytest.mark.parametrize("cols", [96, 4096])
def test_softmax_of_large_magnitudes(mean, std, cols):
    """Row maxima far from zero: the exponent of every term must be taken relative to the maximum without
    losing it to the rounding of a large product (also for rows spread over several warps)."""
    spec = f"hct 1\ninput x f32 [64,{cols}]\nnode p = row_softmax(x)\nnode s = row_sum(p)\noutput p\noutput s\n"
    check_f32(spec, {"x": {"kind": "normal", "mean": mean, "std": std}})


@pytest.mark.parametrize("seed", list(range(60)))
def test_grown_graphs_reduced_rows(seed):
    """Branching multi-output graphs grown with the whole of Algorithm 1 (usage caps, random connections,
    branches, merges), 96 rows each; every output is compared."""
    spec, laws, _ = sweep.get_grown(seed, rows=96)
    check_f32(spec, laws, seed)


def test_run_twice_is_bitwise_repeatable():
    import torch
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c2_softmax_layernorm_chain", r=512, c=4096)
    t = configs.draw_inputs(spec, laws, 0)
    g = hct.FusedGraph(spec, 0)
    ins = parity.to_device(spec, t)
    a = g.run(ins)[0].clone()
    b = g.run(ins)[0]
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_bad_pointers_are_rejected_on_the_host():
    import torch
    import paper_2506_10401_b200 as hct
    spec = "hct 1\ninput x f32 [8,64]\nnode y = relu(x)\noutput y\n"
    g = hct.FusedGraph(spec, 0)
    x = torch.zeros(8 * 64 + 4, device="cuda")
    y = torch.zeros(8, 64, device="cuda")
    with pytest.raises(hct.HctError) as e:
        hct.hct_graph_run(g.handle, [x.data_ptr() + 4], [y.data_ptr()])
    assert e.value.code == hct.HCT_ERR_INVALID_ARG
    with pytest.raises(hct.HctError):
        hct.hct_graph_run(g.handle, [x.data_ptr()], [])
    with pytest.raises(hct.HctError):
        hct.hct_graph_run(g.handle, [0], [y.data_ptr()])


def test_softmax_feeding_layernorm_uses_known_mean_and_matches():
    spec = """hct 1
input x f32 [130,1000]
input g f32 [1000]
input b f32 [1000]
node p = row_softmax(x)
node y = row_layernorm(p, g, b, eps=1e-7)
node q = add(p, 0.001)
node z = row_layernorm(q, g, b, eps=1e-7)
output y
output z
"""
    check_f32(spec, {"x": N_, "g": POS_, "b": N_})


def test_expired_device_wait_is_reported_and_the_device_stays_usable(monkeypatch):
    """A GEMM whose producer never issues its loads: the consumer's bounded wait runs out, the kernel
    ends normally, hct_graph_status reports the timeout, and the next graph runs as usual."""
    import torch
    import paper_2506_10401_b200 as hct
    spec, laws = configs.get_config("c3_gemm_bf16_gelu_residual", m=128, k=128, n=256)
    t = configs.draw_inputs(spec, laws, 0)
    monkeypatch.setenv("HCT_FAULT_NEVER_ARRIVE", "1")
    monkeypatch.setenv("HCT_WAIT_LIMIT", "2000")
    g = hct.FusedGraph(spec, 0)
    monkeypatch.delenv("HCT_FAULT_NEVER_ARRIVE")
    monkeypatch.delenv("HCT_WAIT_LIMIT")
    g.run(parity.to_device(spec, t))
    torch.cuda.synchronize()
    with pytest.raises(hct.HctError) as e:
        g.status()
    assert e.value.code == hct.HCT_ERR_TIMEOUT
    g.status()  # the word was cleared
    check_bf16(spec, laws)
