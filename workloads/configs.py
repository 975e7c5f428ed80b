"""The benchmark chains as operator-DAG spec text plus the recipe for their inputs.

Each entry gives the spec, and per input the sampling law, so that the CUDA
library and the CPU oracle are fed identical seeded tensors.  Input ``i`` of a
config is drawn from stream ``i`` of the config's seed.
"""
from __future__ import annotations

import math

import numpy as np

from .tensors import make_tensor


def _n(std=1.0, mean=0.0):
    return {"kind": "normal", "mean": mean, "std": std}


def _u(lo, hi):
    return {"kind": "uniform", "lo": lo, "hi": hi}


def gemm_bias_relu(m=256, k=256, n=256):
    spec = f"""hct 1
input a    f32 [{m},{k}]
input b    f32 [{k},{n}]
input bias f32 [{n}]
node  t0 = gemm(a, b)
node  t1 = add(t0, bias)
node  t2 = relu(t1)
output t2 f32
"""
    laws = {"a": _u(-1, 1), "b": _u(-1, 1), "bias": _u(-1, 1)}
    return spec, laws


def softmax_layernorm_chain(r=8192, c=4096):
    spec = f"""hct 1
input x     f32 [{r},{c}]
input scale f32 [{c}]
input shift f32 [{c}]
input gamma f32 [{c}]
input beta  f32 [{c}]
node  t0 = mul(x, scale)
node  t1 = add(t0, shift)
node  t2 = gelu_tanh(t1)
node  t3 = row_softmax(t2)
node  t4 = row_layernorm(t3, gamma, beta, eps=1e-5)
output t4 f32
"""
    laws = {"x": _n(), "scale": _n(0.1, 1.0), "shift": _n(0.1), "gamma": _n(0.1, 1.0), "beta": _n(0.1)}
    return spec, laws


def gemm_bf16_gelu_residual(m=8192, k=4096, n=4096):
    spec = f"""hct 1
input x    bf16 [{m},{k}]
input w    bf16 [{k},{n}]
input bias bf16 [{n}]
input r    bf16 [{m},{n}]
node  t0 = gemm(x, w)
node  t1 = add(t0, bias)
node  t2 = gelu_tanh(t1)
node  t3 = add(t2, r)
output t3 bf16
"""
    laws = {"x": _n(), "w": _n(1.0 / math.sqrt(k)), "bias": _n(0.1), "r": _n()}
    return spec, laws


def conv_bn_relu(n=32, c=128, h=56, w=56, k=128, ksize=3, stride=1, pad=1, nhwc=False):
    spec = f"""hct 1
input x     bf16 [{n},{c},{h},{w}]{" nhwc" if nhwc else ""}
input wt    bf16 [{k},{c},{ksize},{ksize}]
input scale f32  [{k},1,1]
input shift f32  [{k},1,1]
node  t0 = conv2d(x, wt, stride={stride}, pad={pad})
node  t1 = mul(t0, scale)
node  t2 = add(t1, shift)
node  t3 = relu(t2)
output t3 bf16
"""
    laws = {"x": _n(), "wt": _n(math.sqrt(2.0 / (c * ksize * ksize))), "scale": _u(0.5, 1.5), "shift": _n(0.1)}
    return spec, laws


def matmul_dropout_mean_softmax(m=8192, k=4096, n=4096, p=0.2, seed=2024):
    """The fused group of the paper's first case study: matrix product, dropout, mean, softmax.

    The mean leaves one value per row, so the closing softmax is identically one; the mean is a second
    output so that the chain's arithmetic (product, mask, scaling, reduction) can be compared."""
    spec = f"""hct 1
input x bf16 [{m},{k}]
input w bf16 [{k},{n}]
node  t0 = gemm(x, w)
node  t1 = dropout(t0, p={p}, seed={seed})
node  t2 = row_mean(t1)
node  t3 = row_softmax(t2)
output t3 f32
output t2 f32
"""
    laws = {"x": _n(), "w": _n(1.0 / math.sqrt(k))}
    return spec, laws


def conv_block(n=32, c=128, h=56, w=56, k=128):
    """Two stacked conv3x3 -> folded batch norm -> ReLU stages (a VGG-style block): the first stage's
    activations are rounded to bf16 and feed the second convolution without leaving the device."""
    spec = f"""hct 1
input x  bf16 [{n},{c},{h},{w}]
input w1 bf16 [{k},{c},3,3]
input s1 f32  [{k},1,1]
input b1 f32  [{k},1,1]
input w2 bf16 [{k},{k},3,3]
input s2 f32  [{k},1,1]
input b2 f32  [{k},1,1]
node  a0 = conv2d(x, w1, stride=1, pad=1)
node  a1 = mul(a0, s1)
node  a2 = add(a1, b1)
node  a3 = relu(a2)
node  a4 = cast_bf16(a3)
node  c0 = conv2d(a4, w2, stride=1, pad=1)
node  c1 = mul(c0, s2)
node  c2 = add(c1, b2)
node  c3 = relu(c2)
output c3 bf16
"""
    laws = {"x": _n(), "w1": _n(math.sqrt(2.0 / (c * 9))), "s1": _u(0.5, 1.5), "b1": _n(0.1),
            "w2": _n(math.sqrt(2.0 / (k * 9))), "s2": _u(0.5, 1.5), "b2": _n(0.1)}
    return spec, laws


def dwconv_bn_relu(n=32, c=192, h=56, w=56, stride=1):
    """Depthwise conv3x3 -> folded batch norm -> ReLU (the memory-bound stage of a MobileNetV2-style block)."""
    spec = f"""hct 1
input x     bf16 [{n},{c},{h},{w}]
input wt    bf16 [{c},1,3,3]
input scale f32  [{c},1,1]
input shift f32  [{c},1,1]
node  t0 = conv2d(x, wt, stride={stride}, pad=1, groups={c})
node  t1 = mul(t0, scale)
node  t2 = add(t1, shift)
node  t3 = relu(t2)
output t3 bf16
"""
    laws = {"x": _n(), "wt": _n(math.sqrt(2.0 / 9)), "scale": _u(0.5, 1.5), "shift": _n(0.1)}
    return spec, laws


def mbconv_block(n=32, c=32, h=56, w=56, expand=6):
    """An inverted-residual block in the style of MobileNetV2: pointwise expansion -> BN -> ReLU, depthwise
    3x3 -> BN -> ReLU, pointwise projection -> BN, plus the block input; activations between the
    convolutions are rounded to bf16 and stay on the device."""
    e = c * expand
    spec = f"""hct 1
input x  bf16 [{n},{c},{h},{w}]
input w1 bf16 [{e},{c},1,1]
input s1 f32  [{e},1,1]
input b1 f32  [{e},1,1]
input w2 bf16 [{e},1,3,3]
input s2 f32  [{e},1,1]
input b2 f32  [{e},1,1]
input w3 bf16 [{c},{e},1,1]
input s3 f32  [{c},1,1]
input b3 f32  [{c},1,1]
node  a0 = conv2d(x, w1)
node  a1 = mul(a0, s1)
node  a2 = add(a1, b1)
node  a3 = relu(a2)
node  a4 = cast_bf16(a3)
node  d0 = conv2d(a4, w2, pad=1, groups={e})
node  d1 = mul(d0, s2)
node  d2 = add(d1, b2)
node  d3 = relu(d2)
node  d4 = cast_bf16(d3)
node  p0 = conv2d(d4, w3)
node  p1 = mul(p0, s3)
node  p2 = add(p1, b3)
node  y  = add(p2, x)
output y bf16
"""
    laws = {"x": _n(), "w1": _n(math.sqrt(2.0 / c)), "s1": _u(0.5, 1.5), "b1": _n(0.1),
            "w2": _n(math.sqrt(2.0 / 9)), "s2": _u(0.5, 1.5), "b2": _n(0.1),
            "w3": _n(math.sqrt(1.0 / e)), "s3": _u(0.5, 1.5), "b3": _n(0.1)}
    return spec, laws


def mobilenet_stage(n=32, c=32, h=56, w=56, expand=6, blocks=3, c_out=64):
    """Several inverted-residual blocks in a row, as one graph (MobileNetV2 repeats its block within a stage and changes
    resolution and width between stages): `blocks` - 1 blocks of `c` channels at stride 1 with their residuals, then a
    block whose depthwise convolution has stride 2 and whose projection gives `c_out` channels, without a residual.
    Every activation between two convolutions is rounded to bf16 and stays on the device."""
    e = c * expand
    lines = ["hct 1", f"input x bf16 [{n},{c},{h},{w}]"]
    laws = {"x": _n()}
    nodes = []
    cur = "x"
    for i in range(blocks):
        last = i == blocks - 1
        co = c_out if last else c
        for nm, shp, law in ((f"w1_{i}", f"[{e},{c},1,1]", _n(math.sqrt(2.0 / c))), (f"s1_{i}", f"[{e},1,1]", _u(0.5, 1.5)), (f"b1_{i}", f"[{e},1,1]", _n(0.1)),
                             (f"w2_{i}", f"[{e},1,3,3]", _n(math.sqrt(2.0 / 9))), (f"s2_{i}", f"[{e},1,1]", _u(0.5, 1.5)), (f"b2_{i}", f"[{e},1,1]", _n(0.1)),
                             (f"w3_{i}", f"[{co},{e},1,1]", _n(math.sqrt(1.0 / e))), (f"s3_{i}", f"[{co},1,1]", _u(0.5, 1.5)), (f"b3_{i}", f"[{co},1,1]", _n(0.1))):
            lines.append(f"input {nm} {'bf16' if nm[0] == 'w' else 'f32'} {shp}")
            laws[nm] = law
        nodes += [f"node a0_{i} = conv2d({cur}, w1_{i})", f"node a1_{i} = mul(a0_{i}, s1_{i})", f"node a2_{i} = add(a1_{i}, b1_{i})",
                  f"node a3_{i} = relu(a2_{i})", f"node a4_{i} = cast_bf16(a3_{i})",
                  f"node d0_{i} = conv2d(a4_{i}, w2_{i}, stride={2 if last else 1}, pad=1, groups={e})", f"node d1_{i} = mul(d0_{i}, s2_{i})",
                  f"node d2_{i} = add(d1_{i}, b2_{i})", f"node d3_{i} = relu(d2_{i})", f"node d4_{i} = cast_bf16(d3_{i})",
                  f"node p0_{i} = conv2d(d4_{i}, w3_{i})", f"node p1_{i} = mul(p0_{i}, s3_{i})", f"node p2_{i} = add(p1_{i}, b3_{i})"]
        if last:
            nodes.append(f"node y = cast_bf16(p2_{i})")
        else:
            nodes += [f"node r_{i} = add(p2_{i}, {cur})", f"node o_{i} = cast_bf16(r_{i})"]
            cur = f"o_{i}"
    return "\n".join(lines + nodes + ["output y bf16"]) + "\n", laws


def resnext_block(n=32, c=256, h=28, w=28, width=128, groups=32):
    """A bottleneck block with a grouped 3x3 convolution in the style of ResNeXt: 1x1 to `width` channels -> BN -> ReLU,
    3x3 with `groups` groups -> BN -> ReLU, 1x1 back to `c` channels -> BN, plus the block input, ReLU."""
    spec = f"""hct 1
input x  bf16 [{n},{c},{h},{w}]
input w1 bf16 [{width},{c},1,1]
input s1 f32  [{width},1,1]
input b1 f32  [{width},1,1]
input w2 bf16 [{width},{width // groups},3,3]
input s2 f32  [{width},1,1]
input b2 f32  [{width},1,1]
input w3 bf16 [{c},{width},1,1]
input s3 f32  [{c},1,1]
input b3 f32  [{c},1,1]
node  a0 = conv2d(x, w1)
node  a1 = mul(a0, s1)
node  a2 = add(a1, b1)
node  a3 = relu(a2)
node  a4 = cast_bf16(a3)
node  g0 = conv2d(a4, w2, pad=1, groups={groups})
node  g1 = mul(g0, s2)
node  g2 = add(g1, b2)
node  g3 = relu(g2)
node  g4 = cast_bf16(g3)
node  p0 = conv2d(g4, w3)
node  p1 = mul(p0, s3)
node  p2 = add(p1, b3)
node  p3 = add(p2, x)
node  y  = relu(p3)
output y bf16
"""
    laws = {"x": _n(), "w1": _n(math.sqrt(2.0 / c)), "s1": _u(0.5, 1.5), "b1": _n(0.1),
            "w2": _n(math.sqrt(2.0 / (9 * (width // groups)))), "s2": _u(0.5, 1.5), "b2": _n(0.1),
            "w3": _n(math.sqrt(1.0 / width)), "s3": _u(0.5, 1.5), "b3": _n(0.1)}
    return spec, laws


def topk_bias_relu(r=8192, c=4096, k=32):
    """A logic-intensive operator with fused consumers (Table 1): the k largest values of every row, plus a bias, through ReLU."""
    spec = f"""hct 1
input x    f32 [{r},{c}]
input bias f32 [{k}]
node  t0 = row_topk(x, k={k})
node  t1 = add(t0, bias)
node  t2 = relu(t1)
output t2 f32
"""
    laws = {"x": _n(), "bias": _n()}
    return spec, laws


def sort_bias_relu(r=8192, c=4096):
    """The other logic-intensive operator of Table 1 with fused consumers: every row sorted in ascending order, plus a bias, through ReLU."""
    spec = f"""hct 1
input x    f32 [{r},{c}]
input bias f32 [{c}]
node  t0 = row_sort(x)
node  t1 = add(t0, bias)
node  t2 = relu(t1)
output t2 f32
"""
    laws = {"x": _n(), "bias": _n()}
    return spec, laws


def transpose_bias_relu(r=16384, c=4096):
    """A layout transform with fused consumers (Table 1, "LayoutTransform"): y = relu(x^T + bias)."""
    spec = f"""hct 1
input x    f32 [{r},{c}]
input bias f32 [{r}]
node  t0 = transpose(x)
node  t1 = add(t0, bias)
node  t2 = relu(t1)
output t2 f32
"""
    laws = {"x": _n(), "bias": _n()}
    return spec, laws


CONFIGS = {
    "c1_gemm_bias_relu_f32": (gemm_bias_relu, {}),
    "c2_softmax_layernorm_chain": (softmax_layernorm_chain, {}),
    "c3_gemm_bf16_gelu_residual": (gemm_bf16_gelu_residual, {}),
    "c4_conv_bn_relu_bf16": (conv_bn_relu, {}),
    # a ResNet-style downsampling convolution, [32,128,56,56] -> 256 channels at stride 2, activations NCHW / channels-last
    "conv_s2_bn_relu": (conv_bn_relu, dict(k=256, stride=2)),
    "conv_s2_bn_relu_nhwc": (conv_bn_relu, dict(k=256, stride=2, nhwc=True)),
    "matmul_dropout_mean_softmax": (matmul_dropout_mean_softmax, {}),
    "transpose_bias_relu": (transpose_bias_relu, {}),
    "conv_block": (conv_block, {}),
    "dwconv_bn_relu": (dwconv_bn_relu, {}),
    "topk_bias_relu": (topk_bias_relu, {}),
    "sort_bias_relu": (sort_bias_relu, {}),
    "mbconv_block": (mbconv_block, {}),
    "mobilenet_stage": (mobilenet_stage, {}),
    "resnext_block": (resnext_block, {}),
}


def parse_inputs(spec: str):
    """(name, dtype, shape) of every ``input`` line, in order.  Text handling only."""
    out = []
    for line in spec.splitlines():
        line = line.split("#", 1)[0].strip()
        if line.startswith("input"):
            _, name, dtype, shape = line.split(None, 3)
            shape = shape[:shape.index("]") + 1]
            dims = tuple(int(t) for t in shape.strip()[1:-1].split(",") if t.strip())
            out.append((name, dtype, dims))
    return out


def input_layouts(spec: str):
    """name -> "nhwc" for the inputs declared channels-last.  Text handling only."""
    out = {}
    for line in spec.splitlines():
        line = line.split("#", 1)[0].strip()
        if line.startswith("input") and line.endswith("nhwc"):
            out[line.split()[1]] = "nhwc"
    return out


def draw_inputs(spec: str, laws: dict, seed: int = 0) -> dict:
    """name -> array (float32, or uint16 bfloat16 patterns) for every input of ``spec``."""
    tensors = {}
    for stream, (name, dtype, dims) in enumerate(parse_inputs(spec)):
        tensors[name] = make_tensor(laws[name], dims, dtype, seed, stream)
    return tensors


def get_config(name: str, **overrides):
    fn, kw = CONFIGS[name]
    args = dict(kw)
    args.update(overrides)
    return fn(**args)
