"""Pins for the CPU oracle: hand-derived cases, closed forms, brute-force loops written
from the operator definitions, and torch float64 library routines.  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import interp

HERE = os.path.dirname(os.path.abspath(__file__))
RNG = np.random.default_rng(1234)


# ---------------------------------------------------------------- hand-derived fixture file

def _value(tok):
    return float(eval(tok, {"__builtins__": {}}, {"ln": math.log, "sqrt": math.sqrt}))


def _hand_cases():
    cases, cur = [], None
    with open(os.path.join(HERE, "golden", "hand_cases.txt")) as f:
        for raw in f:
            line = raw.rstrip("\n")
            if cur is not None and cur["in_spec"]:
                if line.strip() == "end":
                    cur["in_spec"] = False
                else:
                    cur["spec"].append(line)
                continue
            s = line.split("#", 1)[0].strip()
            if not s:
                continue
            toks = s.split()
            if toks[0] == "case":
                cur = {"name": toks[1], "spec": [], "in_spec": True, "in": {}, "out": {}}
                cases.append(cur)
            elif toks[0] in ("in", "out"):
                cur[toks[0]][toks[1]] = [_value(t) for t in toks[2:]]
    return cases


@pytest.mark.parametrize("case", _hand_cases(), ids=lambda c: c["name"])
def test_hand_cases(case):
    spec = "\n".join(case["spec"])
    g = oracle.parse(spec)
    ins = {n: np.array(v).reshape(g.nodes[n].shape) for n, v in case["in"].items()}
    vals = oracle.run_nodes(g, ins)
    for name, want in case["out"].items():
        got = vals[name].ravel()
        np.testing.assert_allclose(got, np.array(want), rtol=1e-14, atol=1e-14)


# ---------------------------------------------------------------- elementwise

def test_elementwise_identities():
    x = RNG.normal(size=(7, 13)) * 3
    np.testing.assert_array_equal(interp.relu(interp.relu(x)), interp.relu(x))
    assert (interp.relu(x) >= 0).all() and (interp.relu(x)[x > 0] == x[x > 0]).all()
    np.testing.assert_allclose(interp.sigmoid(x) + interp.sigmoid(-x), 1.0, rtol=0, atol=1e-15)
    np.testing.assert_allclose(interp.gelu_tanh(x) - interp.gelu_tanh(-x), x, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(interp.gelu_erf(x) - interp.gelu_erf(-x), x, rtol=1e-14, atol=1e-15)
    assert interp.sigmoid(np.zeros(1))[0] == 0.5


def test_gelu_points_against_scalar_formula():
    for v in (-3.0, -1.0, -0.25, 0.0, 0.5, 1.0, 2.5):
        want_t = 0.5 * v * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (v + 0.044715 * v ** 3)))
        want_e = 0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0)))
        assert abs(interp.gelu_tanh(np.array([v]))[0] - want_t) <= 1e-15
        assert abs(interp.gelu_erf(np.array([v]))[0] - want_e) <= 1e-15
    # the two variants differ visibly, so a swap is caught
    assert abs(interp.gelu_tanh(np.array([2.0]))[0] - interp.gelu_erf(np.array([2.0]))[0]) > 5e-5


def test_elementwise_against_torch64():
    x = RNG.normal(size=(5, 9)) * 2
    t = torch.from_numpy(x)
    np.testing.assert_allclose(interp.gelu_tanh(x), torch.nn.functional.gelu(t, approximate="tanh").numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(interp.gelu_erf(x), torch.nn.functional.gelu(t).numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(interp.sigmoid(x), torch.sigmoid(t).numpy(), rtol=1e-13)


def _spec1(op, shape="[3,4]"):
    return f"hct 1\ninput x f32 {shape}\nnode y = {op}(x)\noutput y\n"


@pytest.mark.parametrize("op,fn", [("exp", math.exp), ("tanh", math.tanh), ("sin", math.sin), ("cos", math.cos),
                                   ("neg", lambda v: -v), ("abs", abs), ("sqrt", lambda v: math.sqrt(v)), ("log", math.log),
                                   ("rsqrt", lambda v: 1.0 / math.sqrt(v)), ("square", lambda v: v * v), ("reciprocal", lambda v: 1.0 / v)])
def test_unary_through_interpreter(op, fn):
    x = np.abs(RNG.normal(size=(3, 4))) + 0.1 if op in ("sqrt", "log", "rsqrt", "reciprocal") else RNG.normal(size=(3, 4))
    y = oracle.run(_spec1(op), {"x": x})["y"]
    want = np.array([[fn(v) for v in row] for row in x])
    np.testing.assert_allclose(y, want, rtol=1e-15, atol=0)


@pytest.mark.parametrize("op,fn", [("add", lambda a, b: a + b), ("sub", lambda a, b: a - b), ("mul", lambda a, b: a * b),
                                   ("div", lambda a, b: a / b), ("max", max), ("min", min)])
def test_binary_broadcast_kinds_bruteforce(op, fn):
    r, c = 3, 5
    x = RNG.normal(size=(r, c))
    full = RNG.normal(size=(r, c)) + 3
    rowv = RNG.normal(size=(c,)) + 3
    colv = RNG.normal(size=(r, 1)) + 3
    spec = f"""hct 1
input x f32 [{r},{c}]
input full f32 [{r},{c}]
input rowv f32 [{c}]
input colv f32 [{r},1]
node a = {op}(x, full)
node b = {op}(x, rowv)
node c = {op}(x, colv)
node d = {op}(x, 2.5)
node e = {op}(2.5, x)
node f = {op}(rowv, x)
output a
output b
output c
output d
output e
output f
"""
    out = oracle.run(spec, {"x": x, "full": full, "rowv": rowv, "colv": colv})
    for i in range(r):
        for j in range(c):
            assert out["a"][i, j] == fn(x[i, j], full[i, j])
            assert out["b"][i, j] == fn(x[i, j], rowv[j])
            assert out["c"][i, j] == fn(x[i, j], colv[i, 0])
            assert out["d"][i, j] == fn(x[i, j], 2.5)
            assert out["e"][i, j] == fn(2.5, x[i, j])
            assert out["f"][i, j] == fn(rowv[j], x[i, j])


def test_channel_broadcast_bruteforce():
    x = RNG.normal(size=(2, 3, 2, 2))
    s = RNG.normal(size=(3, 1, 1))
    spec = "hct 1\ninput x f32 [2,3,2,2]\ninput s f32 [3,1,1]\nnode y = mul(x, s)\noutput y\n"
    y = oracle.run(spec, {"x": x, "s": s})["y"]
    for n in range(2):
        for k in range(3):
            for h in range(2):
                for w in range(2):
                    assert y[n, k, h, w] == x[n, k, h, w] * s[k, 0, 0]


# ---------------------------------------------------------------- row reductions

def test_softmax_closed_forms():
    x = RNG.normal(size=(6, 37)) * 4
    y = interp.row_softmax(x)
    np.testing.assert_allclose(y.sum(axis=1), 1.0, rtol=0, atol=1e-12)
    assert (y > 0).all()
    shift = RNG.normal(size=(6, 1)) * 50
    np.testing.assert_allclose(interp.row_softmax(x + shift), y, rtol=1e-12)
    np.testing.assert_allclose(interp.row_softmax(np.full((2, 8), 3.25)), 1.0 / 8, rtol=1e-15)
    # large arguments must not overflow (max subtraction)
    big = np.array([[1000.0, 1000.0 + math.log(3.0)]])
    np.testing.assert_allclose(interp.row_softmax(big), [[0.25, 0.75]], rtol=1e-12)


def test_softmax_bruteforce_and_torch():
    x = RNG.normal(size=(4, 11)) * 2
    y = interp.row_softmax(x)
    for i in range(4):
        m = max(x[i])
        den = sum(math.exp(v - m) for v in x[i])
        for j in range(11):
            assert abs(y[i, j] - math.exp(x[i, j] - m) / den) <= 1e-15
    np.testing.assert_allclose(y, torch.softmax(torch.from_numpy(x), dim=1).numpy(), rtol=1e-12)


def test_row_sum_mean_max_bruteforce():
    x = RNG.normal(size=(5, 17))
    s, m, mx = interp.row_sum(x), interp.row_mean(x), interp.row_max(x)
    assert s.shape == m.shape == mx.shape == (5, 1)
    for i in range(5):
        assert abs(s[i, 0] - math.fsum(x[i])) <= 1e-14
        assert abs(m[i, 0] - math.fsum(x[i]) / 17) <= 1e-15
        assert mx[i, 0] == max(x[i])


def test_layernorm_closed_forms():
    c = 64
    x = RNG.normal(size=(5, c)) * 0.01 + 2.0
    ones, zeros = np.ones(c), np.zeros(c)
    for eps in (0.0, 1e-5, 1e-2):
        y = interp.row_layernorm(x, ones, zeros, eps)
        v = x.var(axis=1)  # numpy's default is the biased variance
        np.testing.assert_allclose(y.mean(axis=1), 0.0, atol=1e-12)
        np.testing.assert_allclose(y.var(axis=1), v / (v + eps), rtol=1e-10)
    gamma, beta = RNG.normal(size=c), RNG.normal(size=c)
    yhat = interp.row_layernorm(x, ones, zeros, 1e-5)
    np.testing.assert_allclose(interp.row_layernorm(x, gamma, beta, 1e-5), yhat * gamma + beta, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(interp.row_layernorm(np.full((2, c), 7.0), gamma, beta, 1e-5), np.tile(beta, (2, 1)), atol=1e-15)


def test_layernorm_bruteforce_and_torch():
    r, c, eps = 3, 10, 1e-3
    x, gamma, beta = RNG.normal(size=(r, c)), RNG.normal(size=c), RNG.normal(size=c)
    y = interp.row_layernorm(x, gamma, beta, eps)
    for i in range(r):
        mu = math.fsum(x[i]) / c
        var = math.fsum((v - mu) ** 2 for v in x[i]) / c
        for j in range(c):
            want = (x[i, j] - mu) / math.sqrt(var + eps) * gamma[j] + beta[j]
            assert abs(y[i, j] - want) <= 1e-14
    t = torch.nn.functional.layer_norm(torch.from_numpy(x), (c,), torch.from_numpy(gamma), torch.from_numpy(beta), eps)
    np.testing.assert_allclose(y, t.numpy(), rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- gemm

def test_gemm_structure_pins():
    a = RNG.normal(size=(5, 7))
    np.testing.assert_array_equal(interp.gemm(a, np.eye(7)), a)
    sel = np.zeros((7, 2)); sel[3, 0] = 1; sel[6, 1] = 1
    np.testing.assert_array_equal(interp.gemm(a, sel), a[:, [3, 6]])
    np.testing.assert_allclose(interp.gemm(a, np.ones((7, 1))), interp.row_sum(a), rtol=1e-14)
    # non-square, non-symmetric: a transposed operand or swapped order cannot pass
    b = RNG.normal(size=(7, 3))
    c = interp.gemm(a, b)
    assert c.shape == (5, 3)
    for i in range(5):
        for j in range(3):
            assert abs(c[i, j] - math.fsum(a[i, k] * b[k, j] for k in range(7))) <= 1e-14
    # square, non-symmetric B = [[0,1],[0,0]] shifts columns right: [a0,a1] -> [0,a0]
    sq = interp.gemm(np.array([[2.0, 3.0], [5.0, 7.0]]), np.array([[0.0, 1.0], [0.0, 0.0]]))
    np.testing.assert_array_equal(sq, [[0.0, 2.0], [0.0, 5.0]])


def test_gemm_integer_exact_and_torch():
    a = RNG.integers(-8, 9, size=(33, 65)).astype(np.float64)
    b = RNG.integers(-8, 9, size=(65, 17)).astype(np.float64)
    want = (a.astype(np.int64) @ b.astype(np.int64)).astype(np.float64)
    np.testing.assert_array_equal(interp.gemm(a, b), want)
    x, y = RNG.normal(size=(12, 31)), RNG.normal(size=(31, 9))
    np.testing.assert_allclose(interp.gemm(x, y), torch.matmul(torch.from_numpy(x), torch.from_numpy(y)).numpy(), rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- conv2d

def _conv_loops(x, w, stride, pad, dil=1, groups=1):
    """The definition as a seven-deep loop nest (NCHW, zero contribution outside the image)."""
    n_, _, h_, w_ = x.shape
    k_, c_, r_, s_ = w.shape            # c_ channels per group
    ho = (h_ + 2 * pad - dil * (r_ - 1) - 1) // stride + 1
    wo = (w_ + 2 * pad - dil * (s_ - 1) - 1) // stride + 1
    y = np.zeros((n_, k_, ho, wo))
    for n in range(n_):
        for k in range(k_):
            for h in range(ho):
                for q in range(wo):
                    acc = 0.0
                    for c in range(c_):
                        for r in range(r_):
                            for s in range(s_):
                                ih = h * stride - pad + r * dil
                                iw = q * stride - pad + s * dil
                                if 0 <= ih < h_ and 0 <= iw < w_:
                                    acc += x[n, (k // (k_ // groups)) * c_ + c, ih, iw] * w[k, c, r, s]
                    y[n, k, h, q] = acc
    return y


@pytest.mark.parametrize("shape,wshape,stride,pad", [
    ((2, 3, 5, 6), (4, 3, 3, 3), 1, 1),
    ((1, 2, 7, 5), (3, 2, 3, 3), 2, 1),
    ((1, 2, 6, 6), (2, 2, 2, 3), 1, 0),
    ((2, 1, 4, 4), (2, 1, 3, 3), 1, 2),
    ((1, 3, 5, 5), (2, 3, 1, 1), 2, 0),
])
def test_conv_bruteforce_and_torch(shape, wshape, stride, pad):
    x, w = RNG.normal(size=shape), RNG.normal(size=wshape)
    y = interp.conv2d(x, w, stride, pad)
    np.testing.assert_allclose(y, _conv_loops(x, w, stride, pad), rtol=1e-13, atol=1e-13)
    t = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(w), stride=stride, padding=pad)
    np.testing.assert_allclose(y, t.numpy(), rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("shape,wshape,stride,pad,dil", [
    ((1, 2, 9, 8), (3, 2, 3, 3), 1, 2, 2),
    ((2, 1, 11, 10), (2, 1, 3, 2), 2, 1, 3),
    ((1, 3, 7, 7), (2, 3, 2, 2), 1, 0, 2),
])
def test_conv_dilation_bruteforce_and_torch(shape, wshape, stride, pad, dil):
    x, w = RNG.normal(size=shape), RNG.normal(size=wshape)
    y = interp.conv2d(x, w, stride, pad, dil)
    np.testing.assert_allclose(y, _conv_loops(x, w, stride, pad, dil), rtol=1e-13, atol=1e-13)
    t = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(w), stride=stride, padding=pad, dilation=dil)
    np.testing.assert_allclose(y, t.numpy(), rtol=1e-12, atol=1e-12)
    # a dilated filter equals the dense filter with zeros between its taps
    k_, c_, r_, s_ = wshape
    wz = np.zeros((k_, c_, dil * (r_ - 1) + 1, dil * (s_ - 1) + 1))
    wz[:, :, ::dil, ::dil] = w
    np.testing.assert_allclose(y, interp.conv2d(x, wz, stride, pad), rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("shape,wshape,stride,pad,dil,groups", [
    ((2, 6, 7, 8), (6, 1, 3, 3), 1, 1, 1, 6),        # depthwise
    ((1, 4, 9, 9), (8, 1, 3, 3), 2, 1, 1, 4),        # depthwise, two filters per channel
    ((1, 6, 8, 7), (4, 3, 3, 2), 1, 1, 2, 2),
    ((2, 8, 6, 6), (12, 2, 1, 1), 1, 0, 1, 4),
])
def test_conv_groups_bruteforce_torch_and_block_diagonal(shape, wshape, stride, pad, dil, groups):
    x, w = RNG.normal(size=shape), RNG.normal(size=wshape)
    y = interp.conv2d(x, w, stride, pad, dil, groups)
    np.testing.assert_allclose(y, _conv_loops(x, w, stride, pad, dil, groups), rtol=1e-13, atol=1e-13)
    t = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(w), stride=stride, padding=pad, dilation=dil, groups=groups)
    np.testing.assert_allclose(y, t.numpy(), rtol=1e-12, atol=1e-12)
    # a grouped filter bank is a dense one whose weights vanish outside the diagonal blocks
    k_, cg, r_, s_ = wshape
    dense = np.zeros((k_, cg * groups, r_, s_))
    for k in range(k_):
        g = k // (k_ // groups)
        dense[k, g * cg:(g + 1) * cg] = w[k]
    np.testing.assert_allclose(y, interp.conv2d(x, dense, stride, pad, dil), rtol=1e-13, atol=1e-13)


def test_conv_structure_pins():
    n, c, h, w, k = 2, 3, 5, 4, 4
    x = RNG.normal(size=(n, c, h, w))
    # 1x1 filter == GEMM over channels
    w1 = RNG.normal(size=(k, c, 1, 1))
    y = interp.conv2d(x, w1, 1, 0)
    want = np.einsum("nchw,kc->nkhw", x, w1[:, :, 0, 0])
    np.testing.assert_allclose(y, want, rtol=1e-13, atol=1e-14)
    # centre-tap delta filter is the identity
    wd = np.zeros((c, c, 3, 3))
    for i in range(c):
        wd[i, i, 1, 1] = 1.0
    np.testing.assert_array_equal(interp.conv2d(x, wd, 1, 1), x)
    # all-ones input and filter count the taps inside the image: 9C interior, 6C edges, 4C corners
    y1 = interp.conv2d(np.ones((1, c, 5, 5)), np.ones((1, c, 3, 3)), 1, 1)[0, 0]
    assert y1[2, 2] == 9 * c and y1[0, 2] == 6 * c and y1[2, 0] == 6 * c and y1[0, 0] == 4 * c and y1[4, 4] == 4 * c
    # integer inputs give exact results
    xi = RNG.integers(-4, 5, size=(1, 3, 6, 6)).astype(np.float64)
    wi = RNG.integers(-4, 5, size=(2, 3, 3, 3)).astype(np.float64)
    np.testing.assert_array_equal(interp.conv2d(xi, wi, 1, 1), _conv_loops(xi, wi, 1, 1))


# ---------------------------------------------------------------- reshape

def test_reshape_keeps_row_major_order():
    x = np.arange(2 * 3 * 4 * 5, dtype=np.float64).reshape(2, 3, 4, 5)
    y = interp.reshape(x, 6, 20)
    np.testing.assert_array_equal(y.ravel(), np.arange(120))            # element t stays element t
    assert y[4, 7] == x[1, 1, 1, 2]                                     # 4*20+7 = 87 = ((1*3+1)*4+1)*5+2
    for (n, c, h, w) in [(2, 3, 4, 5), (1, 7, 2, 2)]:
        a = RNG.normal(size=(n, c, h, w))
        f = interp.reshape(a, n, c * h * w)
        for i in range(n):
            for j in range(c):
                for k in range(h):
                    for m in range(w):
                        assert f[i, (j * h + k) * w + m] == a[i, j, k, m]
    a = RNG.normal(size=(6, 8))
    np.testing.assert_array_equal(interp.reshape(interp.reshape(a, 12, 4), 6, 8), a)
    g = oracle.parse("hct 1\ninput x bf16 [2,3,4,5]\nnode f = reshape(x, rows=6, cols=20)\noutput f bf16\n")
    assert g.nodes["f"].shape == (6, 20) and g.nodes["f"].dtype == "bf16"
    with pytest.raises(oracle.SpecError):
        oracle.parse("hct 1\ninput x f32 [2,3]\nnode f = reshape(x, rows=4, cols=2)\noutput f\n")


# ---------------------------------------------------------------- row_sort / row_topk

def _insertion_sorted(row):
    out = []
    for v in row:
        i = 0
        while i < len(out) and out[i] <= v:
            i += 1
        out.insert(i, v)
    return out


def test_sort_hand_values_bruteforce_and_invariants():
    x = np.array([[3.0, 1.0, 2.0, 5.0, 4.0], [0.0, -1.0, 7.0, 7.0, 2.0], [1.0, 1.0, 1.0, 0.0, 9.0]])
    np.testing.assert_array_equal(interp.row_sort(x), [[1, 2, 3, 4, 5], [-1, 0, 2, 7, 7], [0, 1, 1, 1, 9]])
    np.testing.assert_array_equal(interp.row_sort(x, descending=True), [[5, 4, 3, 2, 1], [7, 7, 2, 0, -1], [9, 1, 1, 1, 0]])
    np.testing.assert_array_equal(interp.row_topk(x, 2), [[5, 4], [7, 7], [9, 1]])
    y = RNG.integers(-5, 6, size=(7, 23)).astype(np.float64)          # many equal values
    z = RNG.normal(size=(5, 40))
    for a in (y, z):
        s = interp.row_sort(a)
        for i in range(a.shape[0]):
            assert list(s[i]) == _insertion_sorted(list(a[i]))
        assert np.all(np.diff(s, axis=1) >= 0)
        np.testing.assert_array_equal(interp.row_sort(a, descending=True), s[:, ::-1])
        # sorting is invariant under a permutation of the columns and idempotent
        np.testing.assert_array_equal(interp.row_sort(a[:, RNG.permutation(a.shape[1])]), s)
        np.testing.assert_array_equal(interp.row_sort(s), s)
        # top-k by repeatedly removing the maximum
        for k in (1, 3, a.shape[1]):
            t = interp.row_topk(a, k)
            for i in range(a.shape[0]):
                rest, want = list(a[i]), []
                for _ in range(k):
                    m = max(rest)
                    want.append(m)
                    rest.remove(m)
                assert list(t[i]) == want
    g = oracle.parse("hct 1\ninput x f32 [4,9]\nnode t = row_topk(x, k=3)\nnode s = row_sort(x, descending=1)\noutput t\noutput s\n")
    assert g.nodes["t"].shape == (4, 3) and g.nodes["s"].shape == (4, 9)


def test_permute_hand_values_inverse_and_library():
    x = np.arange(24, dtype=np.float64).reshape(2, 3, 4)
    y = interp.permute(x, (2, 0, 1))                       # y[k, i, j] = x[i, j, k]
    assert y.shape == (4, 2, 3)
    assert y[3, 1, 2] == x[1, 2, 3] == 23 and y[1, 0, 2] == x[0, 2, 1] == 9 and y[0, 1, 0] == x[1, 0, 0] == 12
    z = RNG.normal(size=(3, 4, 5, 6))
    import itertools
    for axes in itertools.permutations(range(4)):
        p = interp.permute(z, axes)
        np.testing.assert_array_equal(p, np.transpose(z, axes))                      # library routine
        inv = tuple(int(np.argsort(axes)[d]) for d in range(4))
        np.testing.assert_array_equal(interp.permute(p, inv), z)                     # the inverse permutation undoes it
        assert sorted(p.ravel()) == sorted(z.ravel())
    # two axes: the transposition
    m = RNG.normal(size=(5, 7))
    np.testing.assert_array_equal(interp.permute(m, (1, 0)), interp.transpose(m))
    np.testing.assert_array_equal(interp.permute(m, (0, 1)), m)
    g = oracle.parse("hct 1\ninput x f32 [2,3,4,5]\nnode p = permute(x, axes=0231)\noutput p\n")
    assert g.nodes["p"].shape == (2, 4, 5, 3)
    for bad in ("axes=0221", "axes=012", "axes=0234"):
        with pytest.raises(oracle.SpecError):
            oracle.parse(f"hct 1\ninput x f32 [2,3,4,5]\nnode p = permute(x, {bad})\noutput p\n")


def test_argsort_hand_values_bruteforce_and_ties():
    x = np.array([[3.0, 1.0, 2.0, 5.0, 4.0], [0.0, -1.0, 7.0, 7.0, 2.0], [1.0, 1.0, 1.0, -0.0, 0.0]])
    # hand values: equal values keep their column order in BOTH directions
    np.testing.assert_array_equal(interp.row_argsort(x), [[1, 2, 0, 4, 3], [1, 0, 4, 2, 3], [3, 4, 0, 1, 2]])
    np.testing.assert_array_equal(interp.row_argsort(x, descending=True), [[3, 4, 0, 2, 1], [2, 3, 4, 0, 1], [0, 1, 2, 3, 4]])
    np.testing.assert_array_equal(interp.row_topk_indices(x, 2), [[3, 4], [2, 3], [0, 1]])
    y = RNG.integers(-3, 4, size=(6, 29)).astype(np.float64)          # many equal values
    z = RNG.normal(size=(4, 33))
    for a in (y, z):
        for desc in (False, True):
            idx = interp.row_argsort(a, descending=desc).astype(np.int64)
            # a permutation of the columns that puts the values in order ...
            assert all(sorted(idx[i]) == list(range(a.shape[1])) for i in range(a.shape[0]))
            np.testing.assert_array_equal(np.take_along_axis(a, idx, axis=1), interp.row_sort(a, descending=desc))
            # ... and, by brute force, each slot takes the first not yet used column holding the wanted value
            for i in range(a.shape[0]):
                used, want = set(), []
                for v in interp.row_sort(a, descending=desc)[i]:
                    j = next(j for j in range(a.shape[1]) if j not in used and a[i, j] == v)
                    used.add(j)
                    want.append(j)
                assert list(idx[i]) == want
        np.testing.assert_array_equal(interp.row_argsort(a), np.argsort(a + 0.0, axis=1, kind="stable"))   # library routine
        for k in (1, 5, a.shape[1]):
            np.testing.assert_array_equal(interp.row_topk_indices(a, k), interp.row_argsort(a, descending=True)[:, :k])
            np.testing.assert_array_equal(np.take_along_axis(a, interp.row_topk_indices(a, k).astype(np.int64), axis=1), interp.row_topk(a, k))
    g = oracle.parse("hct 1\ninput x f32 [4,9]\nnode t = row_topk_indices(x, k=3)\nnode s = row_argsort(x, descending=1)\noutput t\noutput s\n")
    assert g.nodes["t"].shape == (4, 3) and g.nodes["s"].shape == (4, 9)


# ---------------------------------------------------------------- graph validity (paper section 3.2)

GOOD = "hct 1\ninput x f32 [4,8]\ninput b f32 [8]\nnode t = add(x, b)\nnode y = row_softmax(t)\noutput y\n"


def test_parse_good_and_shapes():
    g = oracle.parse(GOOD)
    assert g.nodes["t"].shape == (4, 8) and g.nodes["y"].shape == (4, 8)
    assert g.inputs == ["x", "b"] and g.outputs == [("y", "f32")]
    g = oracle.parse("hct 1\ninput x bf16 [2,3,8,8]\ninput w bf16 [5,3,3,3]\nnode y = conv2d(x, w, stride=2, pad=1)\noutput y bf16\n")
    assert g.nodes["y"].shape == (2, 5, 4, 4)
    g = oracle.parse("hct 1\ninput x bf16 [2,3,9,8]\ninput w bf16 [5,3,3,3]\nnode y = conv2d(x, w, pad=1, dilation=2)\noutput y bf16\n")
    assert g.nodes["y"].shape == (2, 5, 7, 6)
    g = oracle.parse("hct 1\ninput x bf16 [2,6,9,8]\ninput w bf16 [12,2,3,3]\nnode y = conv2d(x, w, pad=1, groups=3)\noutput y bf16\n")
    assert g.nodes["y"].shape == (2, 12, 9, 8)
    g = oracle.parse("hct 1\ninput x f32 [4,8]\nnode s = row_sum(x)\nnode y = div(x, s)\noutput y\n")
    assert g.nodes["s"].shape == (4, 1) and g.nodes["y"].shape == (4, 8)


@pytest.mark.parametrize("bad", [
    "",
    "hct 2\ninput x f32 [4]\nnode y = relu(x)\noutput y\n",
    "hct 1\ninput x f32 [4,8]\nnode y = relu(z)\noutput y\n",                       # undefined operand (dangling)
    "hct 1\ninput x f32 [4,8]\nnode y = add(y, x)\noutput y\n",                     # self reference (cycle)
    "hct 1\ninput x f32 [4,8]\nnode a = relu(b)\nnode b = relu(a)\noutput b\n",     # forward reference (cycle)
    "hct 1\ninput x f32 [4,8]\ninput v f32 [7]\nnode y = add(x, v)\noutput y\n",    # shapes do not broadcast
    "hct 1\ninput x f32 [4,8]\ninput w f32 [9,3]\nnode y = gemm(x, w)\noutput y\n",  # contraction mismatch
    "hct 1\ninput x f32 [4,8]\ninput w bf16 [8,3]\nnode y = gemm(x, w)\noutput y\n",  # dtype mismatch
    "hct 1\ninput x f32 [4,8]\nnode y = relu(x)\nnode z = exp(x)\noutput y\n",      # z reaches no output
    "hct 1\ninput x f32 [4,8]\ninput u f32 [4,8]\nnode y = relu(x)\noutput y\n",    # unused input
    "hct 1\ninput x f32 [4,8]\nnode y = frobnicate(x)\noutput y\n",
    "hct 1\ninput x f32 [4,8]\nnode y = relu(x)\nnode y = exp(x)\noutput y\n",      # duplicate name
    "hct 1\ninput x f32 [4,8]\nnode s = row_sum(x)\nnode y = row_max(s)\noutput y\n",  # row op on [R,1]
    "hct 1\ninput x f32 [4,8]\nnode y = relu(x)\n",                                 # no output
    "hct 1\ninput x f32 [4,8]\noutput x\n",
    "hct 1\ninput x f32 [4,8]\nnode y = relu(x, x)\noutput y\n",
    "hct 1\ninput x f32 [4,8]\nnode y = add(1.0, 2.0)\noutput y\n",
])
def test_parse_rejects(bad):
    with pytest.raises(oracle.SpecError):
        oracle.parse(bad)


def test_cast_bf16_pins():
    # exactly representable values pass through; ties go to the even neighbour; 8 significant bits remain
    x = np.array([1.0, -2.5, 0.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -7, 3.0e38, -1e-30])
    y = interp.cast_bf16(x)
    assert y[0] == 1.0 and y[1] == -2.5 and y[2] == 0.0
    assert y[3] == 1.0                      # tie between 1 and 1 + 2^-7: even mantissa wins
    assert y[4] == 1.0 + 2.0 ** -6          # tie between 1 + 2^-7 and 1 + 2^-6: even again
    assert y[5] == 1.0 + 2.0 ** -7
    t = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(y, t)
    z = RNG.normal(size=1000) * 10.0 ** RNG.integers(-5, 5, size=1000)
    np.testing.assert_array_equal(interp.cast_bf16(z), torch.tensor(z, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy())
    assert np.all(np.abs(interp.cast_bf16(z) - z) <= np.abs(z) * 2.0 ** -8)
    np.testing.assert_array_equal(interp.cast_bf16(interp.cast_bf16(z)), interp.cast_bf16(z))   # idempotent


def test_transpose_pins():
    x = RNG.normal(size=(5, 9))
    spec = "hct 1\ninput x f32 [5,9]\nnode t = transpose(x)\nnode u = transpose(t)\noutput t\noutput u\n"
    out = oracle.run(spec, {"x": x})
    assert out["t"].shape == (9, 5)
    for i in range(5):
        for j in range(9):
            assert out["t"][j, i] == x[i, j]
    np.testing.assert_array_equal(out["u"], x)                           # an involution
    np.testing.assert_array_equal(out["t"], torch.from_numpy(x).t().numpy())
    # (A B)^T = B^T A^T ties the layout transform to the matrix product
    a, b = RNG.integers(-8, 9, size=(4, 6)).astype(float), RNG.integers(-8, 9, size=(6, 3)).astype(float)
    spec = ("hct 1\ninput a f32 [4,6]\ninput b f32 [6,3]\nnode p = gemm(a, b)\nnode pt = transpose(p)\nnode at = transpose(a)\n"
            "node bt = transpose(b)\nnode q = gemm(bt, at)\noutput pt\noutput q\n")
    out = oracle.run(spec, {"a": a, "b": b})
    np.testing.assert_array_equal(out["pt"], out["q"])


def test_row_min_and_arg_reductions_bruteforce_and_ties():
    x = RNG.normal(size=(7, 13))
    x[2, 4] = x[2, 9] = x[2].max() + 1.0      # a tie for the maximum: the first column wins
    x[5, 0] = x[5, 12] = x[5].min() - 1.0     # a tie for the minimum
    spec = "hct 1\ninput x f32 [7,13]\nnode a = row_argmax(x)\nnode b = row_argmin(x)\nnode c = row_min(x)\noutput a\noutput b\noutput c\n"
    out = oracle.run(spec, {"x": x})
    for i in range(7):
        best_hi = max(range(13), key=lambda j: (x[i, j], -j))
        best_lo = min(range(13), key=lambda j: (x[i, j], j))
        assert out["a"][i, 0] == best_hi and out["b"][i, 0] == best_lo
        assert out["c"][i, 0] == min(x[i, j] for j in range(13))
    assert out["a"][2, 0] == 4 and out["b"][5, 0] == 0
    t = torch.from_numpy(x)
    np.testing.assert_array_equal(out["a"][:, 0], torch.argmax(t, dim=1).numpy())
    # argmax commutes with increasing maps, argmin is the argmax of the negation
    np.testing.assert_array_equal(interp.row_argmax(np.exp(x)), interp.row_argmax(x))
    np.testing.assert_array_equal(interp.row_argmin(x), interp.row_argmax(-x))


# ---------------------------------------------------------------- dropout (counter-based mask)

_M64 = (1 << 64) - 1


def _hash_int(v):
    """The generator's steps on Python integers (arbitrary precision, masked to 64 bits by hand)."""
    h = v & _M64
    h ^= h >> 17
    h ^= (h << 31) & _M64
    h ^= h >> 8
    return h


def _golden_hash_rows():
    rows = []
    with open(os.path.join(HERE, "golden", "dropout_hash.txt")) as f:
        for line in f:
            line = line.split("#", 1)[0].split()
            if line:
                rows.append(tuple(int(t) for t in line))
    return rows


def test_dropout_hash_hand_values():
    # the integer steps reproduce the hand-derived values, and the oracle's mask agrees with them
    for start, h, r in _golden_hash_rows():
        assert _hash_int(start) == h and h % 1000 == r
        for thr in (0, r, r + 1):
            if thr >= 1000:
                continue
            keep = interp.dropout_keep_mask((1,), start, thr / 1000.0)[0]
            assert bool(keep) == (r >= thr)


def test_dropout_mask_bruteforce_including_wraparound():
    # offsets and seeds beyond 2^31 and up to 2^63: the shift by 31 must wrap modulo 2^64
    for seed, shape, p in [(0, (5, 7), 0.3), (12345, (3, 4, 5), 0.5), ((1 << 33) + 5, (9,), 0.25), ((1 << 63) - 4, (2, 6), 0.9), (77, (1, 1), 0.0)]:
        got = interp.dropout_keep_mask(shape, seed, p)
        want = np.array([_hash_int(i + seed) % 1000 >= round(1000 * p) for i in range(int(np.prod(shape)))]).reshape(shape)
        np.testing.assert_array_equal(got, want)


def test_dropout_closed_forms():
    x = RNG.normal(size=(200, 500))
    np.testing.assert_array_equal(interp.dropout(x, 0.0, 9), x)            # p = 0 keeps everything, unscaled
    y = interp.dropout(x, 0.2, 9)
    kept = y != 0.0
    np.testing.assert_allclose(y[kept], x[kept] / 0.8, rtol=1e-15)
    np.testing.assert_array_equal(kept, interp.dropout_keep_mask(x.shape, 9, 0.2))   # mask does not depend on x
    assert abs(kept.mean() - 0.8) < 0.01
    # a row-major reshape moves no element's offset: same mask
    np.testing.assert_array_equal(interp.dropout_keep_mask((100, 1000), 9, 0.2).ravel(), interp.dropout_keep_mask((100000,), 9, 0.2))
    # through the interpreter, in the case-study chain: the closing softmax of one value per row is one
    spec = "hct 1\ninput a f32 [6,8]\ninput b f32 [8,10]\nnode t = gemm(a, b)\nnode d = dropout(t, p=0.3, seed=5)\nnode m = row_mean(d)\nnode s = row_softmax(m)\noutput s\noutput m\n"
    a, b = RNG.normal(size=(6, 8)), RNG.normal(size=(8, 10))
    out = oracle.run(spec, {"a": a, "b": b})
    np.testing.assert_array_equal(out["s"], np.ones((6, 1)))
    t = a @ b
    want = np.array([[sum(t[i, j] / 0.7 for j in range(10) if _hash_int(i * 10 + j + 5) % 1000 >= 300) / 10] for i in range(6)])
    np.testing.assert_allclose(out["m"], want, rtol=1e-13)


# ---------------------------------------------------------------- planted mistakes must be caught

def test_planted_mistakes_are_detected(monkeypatch):
    """Each plausible slip, planted into the oracle, makes at least one pin above fail."""
    import copy

    def fails(check):
        try:
            check()
        except Exception:
            return True
        return False

    orig = copy.copy(interp.__dict__)

    def unbiased_ln(x, g, b, eps):
        mu = x.mean(axis=1, keepdims=True); d = x - mu
        v = (d * d).sum(axis=1, keepdims=True) / (x.shape[1] - 1)
        return d / np.sqrt(v + eps) * g.reshape(1, -1) + b.reshape(1, -1)

    def eps_outside_ln(x, g, b, eps):
        mu = x.mean(axis=1, keepdims=True); d = x - mu
        v = (d * d).mean(axis=1, keepdims=True)
        return d / (np.sqrt(v) + eps) * g.reshape(1, -1) + b.reshape(1, -1)

    def flipped_conv(x, w, stride, pad):
        return orig["conv2d"](x, w[:, :, ::-1, ::-1], stride, pad)

    def transposed_gemm(a, b):
        return np.matmul(a, b.T) if b.shape[0] == b.shape[1] else np.matmul(a, b)

    def softmax_no_max(x):
        e = np.exp(x)
        return e / e.sum(axis=1, keepdims=True)

    def gelu_swapped(x):
        return orig["gelu_erf"](x)

    plants = [
        ("reshape", lambda x, rows, cols: np.ascontiguousarray(x).ravel(order="F").reshape(rows, cols), test_reshape_keeps_row_major_order),
        ("row_sort", lambda x, descending=False: orig["row_sort"](x, not descending), test_sort_hand_values_bruteforce_and_invariants),
        ("row_topk", lambda x, k: orig["row_sort"](x)[:, :k], test_sort_hand_values_bruteforce_and_invariants),
        ("row_argsort", lambda x, descending=False: np.argsort(-x if descending else x, axis=1).astype(np.float64)[:, ::1] if not descending
         else np.argsort(x, axis=1, kind="stable")[:, ::-1].astype(np.float64), test_argsort_hand_values_bruteforce_and_ties),
        ("permute", lambda x, axes: np.transpose(x, tuple(int(v) for v in np.argsort(axes))), test_permute_hand_values_inverse_and_library),
        ("row_layernorm", unbiased_ln, test_layernorm_closed_forms),
        ("row_layernorm", eps_outside_ln, test_layernorm_bruteforce_and_torch),
        ("conv2d", flipped_conv, test_conv_structure_pins),
        ("gemm", transposed_gemm, test_gemm_structure_pins),
        ("gemm", lambda a, b: np.matmul(a[:, :-1], b[:-1]), test_gemm_integer_exact_and_torch),
        ("gelu_tanh", gelu_swapped, test_gelu_points_against_scalar_formula),
    ]
    for name, wrong, check in plants:
        monkeypatch.setattr(interp, name, wrong)
        assert fails(check), f"planted mistake in {name} ({wrong.__name__}) was not detected"
        monkeypatch.setattr(interp, name, orig[name])
        check()
    def mask_32bit(shape, seed, p):   # the shift by 31 truncated to 32 bits
        n = int(np.prod(shape))
        h = (np.arange(n, dtype=np.uint64) + np.uint64(seed))
        h ^= h >> np.uint64(17)
        h ^= (h << np.uint64(31)) & np.uint64(0xffffffff)
        h ^= h >> np.uint64(8)
        return ((h % np.uint64(1000)) >= np.uint64(round(p * 1000.0))).reshape(shape)

    def mask_strict(shape, seed, p):  # keeps only variates strictly above p
        return orig["dropout_keep_mask"](shape, seed, p) & (orig["dropout_keep_mask"](shape, seed, min(p + 0.001, 0.999)) | (p >= 0.999))

    for wrong, check in [(mask_32bit, test_dropout_hash_hand_values), (mask_strict, test_dropout_closed_forms)]:
        monkeypatch.setattr(interp, "dropout_keep_mask", wrong)
        assert fails(check), f"planted mistake {wrong.__name__} was not detected"
        monkeypatch.setattr(interp, "dropout_keep_mask", orig["dropout_keep_mask"])
        check()
    monkeypatch.setattr(interp, "row_softmax", softmax_no_max)
    with np.errstate(over="ignore", invalid="ignore"):
        assert fails(test_softmax_closed_forms)
