"""Pins of the oracle's optional paths against what the paper and the mathematics fix:
the border variant of K, ReLU after BinConv, k-bit activations q_k (Section 3.2, "k-bit
Quantization") and the Binary-Weight-Network convolution (Section 3.1, Eq. 1).

As in test_oracle_pins.py no expected value is the oracle's own formula retyped: library
routines in fp64 (torch), exact rational arithmetic, brute force, special cases in which an
option reduces to an already pinned function, and the paper's printed formula for q_k
evaluated with fractions.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def _valid_taps(H, W, kh, kw, s, p):
    ones = torch.ones(1, 1, H, W, dtype=torch.float64)
    return F.conv2d(ones, torch.ones(1, 1, kh, kw, dtype=torch.float64), stride=s, padding=p)[0, 0].numpy()


# ---------------------------------------------------------------- K, border variant
@pytest.mark.parametrize("kh,kw,stride,pad", [(3, 3, 1, 1), (5, 5, 1, 2), (3, 3, 2, 1),
                                               (2, 4, 1, 1), (7, 7, 1, 3), (1, 1, 2, 0)])
def test_valid_taps_K_matches_library_average_pool(oracle, kh, kw, stride, pad):
    """Mean over the in-image taps = an average pool that does not count padded cells."""
    A = np.abs(rng(131).standard_normal((2, 9, 11))).astype(np.float32)
    K = oracle.box_filter_valid_taps(A, kh, kw, stride, pad)
    ref = F.avg_pool2d(torch.from_numpy(A).double()[:, None], (kh, kw), stride, pad,
                       count_include_pad=False)[:, 0].numpy()
    assert K.shape == ref.shape
    assert np.allclose(K, ref, rtol=1e-6, atol=0)


def test_valid_taps_K_special_cases(oracle):
    A = np.abs(rng(132).standard_normal((2, 6, 5))).astype(np.float32)
    # no padding: every tap is inside, the two variants agree bit for bit
    assert np.array_equal(oracle.box_filter_valid_taps(A, 3, 2, 1, 0), oracle.box_filter(A, 3, 2, 1, 0))
    # with padding they agree in the interior and the variant is larger at the border by
    # exactly kh*kw / valid
    K0, K1 = oracle.box_filter(A, 3, 3, 1, 1), oracle.box_filter_valid_taps(A, 3, 3, 1, 1)
    assert np.array_equal(K0[:, 1:-1, 1:-1], K1[:, 1:-1, 1:-1])
    nv = _valid_taps(6, 5, 3, 3, 1, 1)
    assert np.allclose(K1 * nv[None] / 9.0, K0, rtol=1e-6)
    # constant A: the variant returns the constant everywhere, corners included
    c = np.full((1, 8, 7), 0.5, np.float32)
    assert np.all(oracle.box_filter_valid_taps(c, 5, 3, 1, 2) == 0.5)
    # a window that lies wholly in the padding sees nothing
    K = oracle.box_filter_valid_taps(np.ones((1, 2, 2), np.float32), 1, 1, 1, 1)
    assert K.shape == (1, 4, 4) and K[0, 0, 0] == 0.0 and K[0, 1, 1] == 1.0


@pytest.mark.parametrize("case", [(2, 5, 6, 7, 3, 3, 3, 1, 1), (2, 4, 9, 8, 3, 5, 5, 1, 2),
                                  (2, 6, 9, 10, 4, 3, 3, 2, 1), (1, 33, 5, 4, 2, 3, 2, 1, 1)])
def test_valid_taps_block_is_the_dense_conv_everywhere_for_constant_magnitudes(oracle, case):
    """Eq. 10 with equality (|X_i|, |W_i| constant): with K averaged over the in-image taps the
    block equals the zero-padded dense convolution at the border too."""
    N, C, H, W, Co, kh, kw, s, p = case
    g = rng(3 + sum(case))
    x = np.where(g.random((N, C, H, W)) < 0.5, -0.5, 0.5).astype(np.float32)
    w = np.where(g.random((Co, C, kh, kw)) < 0.5, -0.125, 0.125).astype(np.float32)
    r = oracle.xnor_block_ex(x, w, s, p, k_valid_taps=True)
    dense = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), stride=s, padding=p).numpy()
    assert np.array_equal(r.out.astype(np.float64), dense)
    # and the plain options reproduce the main block
    r0, r1 = oracle.xnor_block(x, w, s, p), oracle.xnor_block_ex(x, w, s, p)
    for name in ("y", "H", "A", "K", "B", "alpha", "acc", "out"):
        assert np.array_equal(getattr(r0, name), getattr(r1, name)), name


# ---------------------------------------------------------------- ReLU
def test_relu_is_max_with_zero(oracle):
    v = np.array([0.0, -0.0, 1e-45, -1e-45, 3.0, -3.0, np.inf, -np.inf], np.float32)
    assert oracle.relu(v).tolist() == [0.0, 0.0, float(np.float32(1e-45)), 0.0, 3.0, 0.0, np.inf, 0.0]
    x = rng(141).standard_normal((2, 3, 5, 4)).astype(np.float32)
    # the already pinned pooling oracle with a 1x1 window and its ReLU switch is the same map
    assert np.array_equal(oracle.relu(x), oracle.maxpool2d(x, 1, 1, 0, relu=True))
    assert np.array_equal(oracle.relu(x), torch.relu(torch.from_numpy(x)).numpy())


def test_relu_block(oracle):
    g = rng(142)
    x = g.standard_normal((2, 6, 7, 8)).astype(np.float32)
    w = g.standard_normal((4, 6, 3, 3)).astype(np.float32)
    res = g.standard_normal((2, 4, 7, 8)).astype(np.float32)
    r0 = oracle.xnor_block(x, w, 1, 1)
    r1 = oracle.xnor_block_ex(x, w, 1, 1, relu=True)
    # K >= 0 and alpha > 0, so without a shortcut ReLU acts on the integer sums alone
    assert np.array_equal(r1.out, oracle.scale_output(np.maximum(r0.acc, 0), r0.K, r0.alpha))
    assert np.array_equal(r1.out, np.maximum(r0.out, 0.0)) and np.array_equal(r1.acc, r0.acc)
    # with a shortcut it follows the addition
    r2 = oracle.xnor_block_ex(x, w, 1, 1, residual=res, relu=True)
    assert np.array_equal(r2.out, np.maximum(oracle.xnor_block(x, w, 1, 1, residual=res).out, 0.0))
    assert (r2.out > 0).any() and (r2.out == 0).any()


# ---------------------------------------------------------------- q_k
def _paper_qk(x, k):
    """The printed formula, 2([(2^k-1)(x+1)/2]/(2^k-1) - 1/2), in exact rational arithmetic
    with round-half-up, on a value already inside [-1, 1]."""
    m = 2 ** k - 1
    t = m * (Fraction(x) + 1) / 2
    idx = (t + Fraction(1, 2)).__floor__()
    return 2 * (Fraction(idx, m) - Fraction(1, 2))


@pytest.mark.parametrize("k", [1, 2, 3, 4, 7])
def test_quantize_k_is_the_printed_formula(oracle, k):
    m = 2 ** k - 1
    x = np.clip(rng(150 + k).standard_normal(4000) * 0.6, -1, 1).astype(np.float32)
    L = oracle.quantize_k(x, k).astype(np.int64)
    checked = 0
    for xv, lv in zip(x.tolist(), L.tolist()):
        t = m * (Fraction(xv) + 1) / 2
        if abs((t - t.__floor__()) - Fraction(1, 2)) < Fraction(1, 10 ** 6):
            continue                    # within rounding of a decision point: covered below
        assert Fraction(lv, m) == _paper_qk(xv, k)
        checked += 1
    assert checked > 3900
    # the codes are exactly the 2^k odd integers, all of them occur
    assert set(L.tolist()) == set(range(-m, m + 1, 2))


@pytest.mark.parametrize("k", [1, 2, 3, 5])
def test_quantize_k_properties(oracle, k):
    m = 2 ** k - 1
    # monotone, clipped outside [-1, 1], every level is a fixed point
    x = np.sort(rng(160 + k).standard_normal(3000).astype(np.float32) * 1.5)
    L = oracle.quantize_k(x, k).astype(np.int64)
    assert np.all(np.diff(L) >= 0)
    assert np.all(L[x >= 1] == m) and np.all(L[x <= -1] == -m)
    levels = np.arange(-m, m + 1, 2)
    assert np.array_equal(oracle.quantize_k((levels / m).astype(np.float32), k), levels.astype(np.int8))
    # error at most half a step (plus the fp32 rounding of the decision point)
    inside = np.abs(x) <= 1
    assert np.all(np.abs(L[inside] / m - x[inside].astype(np.float64)) <= 1.0 / m + 1e-6)
    # ties go up: the decision points themselves, as fp32 values, map to the upper level
    taus = np.array([(2 * j - 1) / m - 1 for j in range(1, m + 1)], dtype=np.float64).astype(np.float32)
    assert np.array_equal(oracle.quantize_k(taus, k).astype(np.int64), np.arange(-m + 2, m + 1, 2))
    below = np.nextafter(taus, np.float32(-2))
    assert np.array_equal(oracle.quantize_k(below, k).astype(np.int64), np.arange(-m, m - 1, 2))


def test_one_bit_quantisation_is_sign(oracle):
    v = np.array([0.0, -0.0, 1e-45, -1e-45, 3.0, -3.0, np.inf, -np.inf, 0.5, -0.5, 1e-9, -1e-9], np.float32)
    assert np.array_equal(oracle.quantize_k(v, 1), oracle.sign(v))
    x = rng(170).standard_normal(5000).astype(np.float32)
    assert np.array_equal(oracle.quantize_k(x, 1), oracle.sign(x))


def test_kbit_block(oracle):
    """q_k in place of sign: the integer sums are the dense convolution of the level codes with
    sign(W) (library, fp64), the output is that sum / (2^k - 1) times K alpha; k = 1 through the
    same path gives the main block."""
    g = rng(171)
    N, C, H, W, Co = 2, 7, 6, 5, 3
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, 3, 3)).astype(np.float32)
    res = g.standard_normal((N, Co, H, W)).astype(np.float32)
    r1 = oracle.xnor_block(x, w, 1, 1, residual=res)
    assert np.array_equal(oracle.scale_output_k(r1.acc, 1, r1.K, r1.alpha, res), r1.out)
    for k in (2, 3):
        m = 2 ** k - 1
        r = oracle.xnor_block_ex(x, w, 1, 1, residual=res, kbits=k)
        assert np.array_equal(r.H, oracle.quantize_k(x, k))
        sw = torch.where(torch.from_numpy(w) >= 0, 1.0, -1.0).double()
        acc = F.conv2d(torch.from_numpy(r.H).double(), sw, padding=1).numpy()
        assert np.array_equal(r.acc.astype(np.float64), acc)
        assert np.array_equal(r.K, r1.K) and np.array_equal(r.A, r1.A)
        want = acc / m * r.K[:, None].astype(np.float64) * r.alpha[None, :, None, None].astype(np.float64) + res
        assert np.allclose(r.out, want, rtol=1e-6, atol=1e-6)
    # inputs that already sit on the levels and constant-magnitude weights: exact dense conv
    k, m = 2, 3
    xl = (g.integers(0, 4, (1, 4, 6, 6)) * 2 - 3).astype(np.float32) / m
    wc = np.where(g.random((2, 4, 3, 3)) < 0.5, -0.25, 0.25).astype(np.float32)
    r = oracle.xnor_block_ex(xl, wc, 1, 0, kbits=2)
    dense = F.conv2d(torch.from_numpy(xl).double(), torch.from_numpy(wc).double()).numpy()
    # K = mean|x| over the window is not 1 here, so compare the integer part and the scaling apart
    assert np.allclose(r.acc / m * 0.25, dense, rtol=1e-6, atol=1e-6)


# ---------------------------------------------------------------- Binary-Weight-Network (Eq. 1)
def test_round_bf16_matches_library(oracle):
    g = rng(180)
    v = np.concatenate([g.standard_normal(5000).astype(np.float32) * 10.0 ** g.integers(-20, 20, 5000),
                        np.array([0.0, -0.0, 1.0, np.inf, -np.inf, 3.3895314e38, 1e-40, -1e-45], np.float32)])
    v = v.astype(np.float32)
    want = torch.from_numpy(v).bfloat16().float().numpy()
    got = oracle.round_bf16(v)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # ties to even on the 16 dropped bits
    tie = np.array([0x3F808000, 0x3F818000], np.uint32).view(np.float32)
    assert oracle.round_bf16(tie).view(np.uint32).tolist() == [0x3F800000, 0x3F820000]


BWN_CASES = [(2, 5, 6, 7, 3, 3, 3, 1, 1), (1, 33, 5, 4, 2, 3, 2, 1, 1), (2, 4, 9, 8, 3, 5, 5, 1, 2),
             (2, 6, 9, 10, 4, 3, 3, 2, 1), (2, 8, 5, 6, 3, 1, 1, 1, 0), (1, 4, 8, 9, 2, 1, 1, 2, 0)]


@pytest.mark.parametrize("case", BWN_CASES)
def test_bwn_conv_matches_library_conv_with_binary_weights(oracle, case):
    """(I (+) B) alpha is the dense zero-padded convolution of I with the filter alpha B."""
    N, C, H, W, Co, kh, kw, s, p = case
    g = rng(190 + sum(case))
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, kh, kw)).astype(np.float32)
    B, alpha = oracle.binarize_weights(w)
    Ho, Wo = (H + 2 * p - kh) // s + 1, (W + 2 * p - kw) // s + 1
    res = g.standard_normal((N, Co, Ho, Wo)).astype(np.float32)
    wt = torch.from_numpy(B).double() * torch.from_numpy(alpha).double()[:, None, None, None]
    ref = F.conv2d(torch.from_numpy(x).double(), wt, stride=s, padding=p).numpy()
    assert np.allclose(oracle.bwn_conv(x, B, alpha, s, p), ref, rtol=1e-6, atol=1e-6)
    assert np.allclose(oracle.bwn_conv(x, B, alpha, s, p, res), ref + res, rtol=1e-6, atol=1e-6)


def test_bwn_conv_special_cases(oracle):
    g = rng(200)
    # weights of constant magnitude: Eq. 1 holds with equality, the result is the dense conv
    x = g.standard_normal((2, 6, 7, 5)).astype(np.float32)
    w = np.where(g.random((3, 6, 3, 3)) < 0.5, -0.25, 0.25).astype(np.float32)
    B, alpha = oracle.binarize_weights(w)
    dense = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), padding=1).numpy()
    assert np.allclose(oracle.bwn_conv(x, B, alpha, 1, 1), dense, rtol=1e-6, atol=1e-6)
    # brute force on a tiny case: every output is the signed sum of the window
    xs = g.standard_normal((1, 2, 3, 3)).astype(np.float32)
    Bs = np.where(g.random((1, 2, 2, 2)) < 0.5, -1, 1).astype(np.int8)
    out = oracle.bwn_conv(xs, Bs, np.array([2.0], np.float32), 1, 0)
    for oy, ox in itertools.product(range(2), range(2)):
        tot = sum(float(xs[0, c, oy + ky, ox + kx]) * int(Bs[0, c, ky, kx])
                  for c in range(2) for ky in range(2) for kx in range(2))
        assert np.isclose(out[0, 0, oy, ox], 2.0 * tot, rtol=1e-6)
    # flipping all weights flips the output; an all-(+1) filter sums the window
    assert np.array_equal(oracle.bwn_conv(xs, -Bs, np.array([2.0], np.float32), 1, 0), -out)
    # inputs that are +-c as well: Eq. 1 and Eq. 11 coincide where no tap is padded
    xc = np.where(g.random((1, 4, 6, 6)) < 0.5, -0.5, 0.5).astype(np.float32)
    wc = np.where(g.random((2, 4, 3, 3)) < 0.5, -0.125, 0.125).astype(np.float32)
    Bc, ac = oracle.binarize_weights(wc)
    assert np.array_equal(oracle.bwn_conv(xc, Bc, ac, 1, 0), oracle.xnor_block(xc, wc, 1, 0).out)


# --------------------------------------------------------------------------- binary gradient
# N, C, H, W, Co, kh, kw, pad
BGRAD_CASES = [(2, 5, 6, 7, 3, 3, 3, 1), (1, 33, 5, 4, 2, 3, 2, 1), (2, 4, 9, 8, 3, 5, 5, 2),
               (2, 8, 5, 6, 3, 1, 1, 0), (3, 6, 7, 7, 4, 3, 3, 0), (1, 3, 6, 5, 2, 3, 3, 2)]


@pytest.mark.parametrize("case", BGRAD_CASES)
def test_binary_gradient_backward_is_the_library_gradient_of_the_binarised_convolution(oracle, case):
    """With the gradient replaced by gmax * sign(g), the result is what automatic differentiation
    gives for conv2d(x, alpha * B) with that upstream gradient (Section 3.2, "Binary Gradient";
    Algorithm 1: the backward pass uses the binarised filters)."""
    N, C, H, W, Co, kh, kw, p = case
    g = rng(300 + sum(case))
    w = g.standard_normal((Co, C, kh, kw)).astype(np.float32)
    B, alpha = oracle.binarize_weights(w)
    Ho, Wo = H + 2 * p - kh + 1, W + 2 * p - kw + 1
    grad = g.standard_normal((N, Co, Ho, Wo)).astype(np.float32)
    grad[0, 0, 0, 0] = 0.0                                            # sign(0) = +1
    gmax, gin = oracle.binary_gradient_backward(grad, B, alpha, p, (H, W))
    assert np.array_equal(gmax, np.abs(grad).reshape(N, -1).max(axis=1))
    x = torch.zeros((N, C, H, W), dtype=torch.float64, requires_grad=True)
    wt = torch.from_numpy(B).double() * torch.from_numpy(alpha).double()[:, None, None, None]
    ghat = torch.from_numpy(np.where(grad >= 0, 1.0, -1.0)) * torch.from_numpy(gmax).double()[:, None, None, None]
    ref, = torch.autograd.grad(F.conv2d(x, wt, padding=p), x, grad_outputs=ghat)
    assert np.allclose(gin, ref.numpy(), rtol=1e-6, atol=1e-6 * float(np.abs(ref.numpy()).max()))


def test_binary_gradient_backward_special_cases(oracle):
    g = rng(310)
    N, C, H, W, Co, k, p = 2, 4, 5, 6, 3, 3, 1
    B = np.where(g.random((Co, C, k, k)) < 0.5, -1, 1).astype(np.int8)
    alpha = np.array([0.5, 2.0, 0.25], np.float32)
    grad = g.standard_normal((N, Co, H, W)).astype(np.float32)
    gmax, gin = oracle.binary_gradient_backward(grad, B, alpha, p, (H, W))
    # the scale is the largest magnitude, not the mean: one large entry sets it alone
    big = grad.copy(); big[1, 2, 3, 3] = -50.0
    gmax_b, gin_b = oracle.binary_gradient_backward(big, B, alpha, p, (H, W))
    assert gmax_b[1] == 50.0 and gmax_b[0] == gmax[0] and np.array_equal(gin_b[0], gin[0])
    # only the signs and the maximum of g matter: same signs, same maximum -> same result
    other = np.sign(grad) * g.random(grad.shape).astype(np.float32) * gmax[:, None, None, None]
    other = np.where(np.abs(grad) == gmax[:, None, None, None], grad, other).astype(np.float32)
    assert np.array_equal(oracle.binary_gradient_backward(other, B, alpha, p, (H, W))[1], gin)
    # scaling g by a power of two scales the result; negating g (no zeros in it) negates it
    assert np.array_equal(oracle.binary_gradient_backward(4 * grad, B, alpha, p, (H, W))[1], 4 * gin)
    assert np.array_equal(oracle.binary_gradient_backward(-grad, B, alpha, p, (H, W))[1], -gin)
    # 1x1 filters, one output channel: gin = gmax alpha B[0][c] sign(g)
    B1 = np.array([1, -1, 1], np.int8).reshape(1, 3, 1, 1)
    g1 = g.standard_normal((1, 1, 4, 4)).astype(np.float32)
    m1, gin1 = oracle.binary_gradient_backward(g1, B1, np.array([0.75], np.float32), 0, (4, 4))
    want = (m1[0] * 0.75) * np.where(g1 >= 0, 1.0, -1.0)[:, 0][:, None] * B1.reshape(1, 3, 1, 1)
    assert np.allclose(gin1, want, rtol=1e-6)
    # brute force on a tiny case, taps that leave the gradient's extent contribute nothing
    Bs = np.where(g.random((2, 1, 2, 2)) < 0.5, -1, 1).astype(np.int8)
    gs = g.standard_normal((1, 2, 3, 3)).astype(np.float32)                 # H = W = 4, k = 2, pad 0
    a2 = np.array([1.0, 3.0], np.float32)
    ms, gins = oracle.binary_gradient_backward(gs, Bs, a2, 0, (4, 4))
    for y, x in itertools.product(range(4), range(4)):
        tot = 0.0
        for co, ky, kx in itertools.product(range(2), range(2), range(2)):
            oy, ox = y - ky, x - kx
            if 0 <= oy < 3 and 0 <= ox < 3:
                tot += float(a2[co]) * int(Bs[co, 0, ky, kx]) * (1.0 if gs[0, co, oy, ox] >= 0 else -1.0)
        assert np.isclose(gins[0, 0, y, x], float(ms[0]) * tot, rtol=1e-6, atol=1e-6)


def test_binary_gradient_backward_product_rounding(oracle):
    """round_products rounds gmax * alpha to bfloat16: no effect when the products are
    representable, otherwise the result is that of the rounded products."""
    g = rng(320)
    B = np.where(g.random((3, 4, 3, 3)) < 0.5, -1, 1).astype(np.int8)
    grad = g.standard_normal((2, 3, 5, 5)).astype(np.float32)
    grad[:, 0, 0, 0] = [4.0, -8.0]                                           # gmax = 4, 8
    exact_alpha = np.array([0.5, 1.25, 3.0], np.float32)
    a = oracle.binary_gradient_backward(grad, B, exact_alpha, 1, (5, 5), round_products=False)[1]
    b = oracle.binary_gradient_backward(grad, B, exact_alpha, 1, (5, 5), round_products=True)[1]
    assert np.array_equal(a, b)
    alpha = np.array([0.3337, 1.2345, 0.071], np.float32)
    r = oracle.binary_gradient_backward(grad, B, alpha, 1, (5, 5), round_products=True)[1]
    for n, m in enumerate((4.0, 8.0)):
        t = oracle.round_bf16((np.float32(m) * alpha).astype(np.float32))
        # the rounded products as the filter scales of an unrounded run with gmax = 1
        unit = np.where(grad[n:n + 1] >= 0, 1.0, -1.0).astype(np.float32)
        want = oracle.binary_gradient_backward(unit, B, t, 1, (5, 5), round_products=False)[1]
        assert np.allclose(r[n:n + 1], want, rtol=1e-6, atol=1e-6)
    assert not np.array_equal(r, oracle.binary_gradient_backward(grad, B, alpha, 1, (5, 5))[1])
