"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests retypes the oracle's own formula as the expected value:
they use brute force over all sign patterns, exact rational arithmetic, a
bit-packed XOR/popcount routine written only here, library convolutions
(torch, fp64) on inputs where the approximation is exact, closed forms and
invariants.  Shapes are deliberately non-square (H != W, kh != kw) so that a
transposed index in the oracle cannot pass.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


# ---------------------------------------------------------------- Eq. 2-6
@pytest.mark.parametrize("n,seed", [(1, 1), (2, 2), (5, 3), (9, 4), (12, 5)])
def test_closed_form_is_the_brute_force_minimum(oracle, n, seed):
    """Eq. 2: (alpha*, B*) minimises ||W - alpha B||^2 over alpha>0, B in {+-1}^n.
    Enumerate every B, use the best alpha for each (Eq. 5), compare."""
    w = rng(seed).standard_normal(n)
    w32 = w.astype(np.float32).reshape(1, n, 1, 1)
    B, alpha = oracle.binarize_weights(w32)
    wd = w32.reshape(-1).astype(np.float64)
    best_J, best_B = None, None
    for pat in itertools.product((-1.0, 1.0), repeat=n):
        b = np.array(pat)
        a = wd @ b / n                      # stationary point of J in alpha for this B
        if a <= 0:
            continue
        J = np.sum((wd - a * b) ** 2)
        if best_J is None or J < best_J:
            best_J, best_B = J, b
    J_oracle = np.sum((wd - float(alpha[0]) * B.reshape(-1)) ** 2)
    assert np.array_equal(best_B, B.reshape(-1).astype(np.float64))
    assert J_oracle <= best_J * (1 + 1e-6) + 1e-12
    # Eq. 3 at the optimum: J* = W^T W - n alpha*^2
    assert np.isclose(J_oracle, wd @ wd - n * float(alpha[0]) ** 2, rtol=1e-5, atol=1e-7)
    # alpha is a strict minimum along alpha for B*
    for d in (1e-2, -1e-2):
        assert np.sum((wd - (alpha[0] + d) * B.reshape(-1)) ** 2) > J_oracle


def test_alpha_is_per_filter_l1_mean(oracle):
    """Eq. 6 with n = c*w*h, one alpha per filter (Section 3.1)."""
    w = rng(7).standard_normal((5, 3, 2, 4)).astype(np.float32)
    B, alpha = oracle.binarize_weights(w)
    exact = [float(sum(Fraction(abs(float(v))) for v in w[co].reshape(-1)) / w[co].size)
             for co in range(5)]
    assert np.allclose(alpha, exact, rtol=1e-7, atol=0)
    assert alpha.shape == (5,)
    # the filters are independent: changing filter 3 moves only alpha[3]
    w2 = w.copy()
    w2[3] *= 3.0
    _, alpha2 = oracle.binarize_weights(w2)
    assert np.array_equal(np.delete(alpha2, 3), np.delete(alpha, 3))
    assert np.isclose(alpha2[3], 3.0 * alpha[3], rtol=1e-6)


def test_sign_convention(oracle):
    """B_i = +1 if W_i >= 0, -1 if W_i < 0 (below Eq. 4); same for inputs."""
    v = np.array([0.0, -0.0, 1e-45, -1e-45, 3.0, -3.0, np.inf, -np.inf, np.nan], np.float32)
    assert oracle.sign(v).tolist() == [1, 1, 1, -1, 1, -1, 1, -1, -1]
    B, _ = oracle.binarize_weights(v[:8].reshape(1, 8, 1, 1))
    assert B.reshape(-1).tolist() == [1, 1, 1, -1, 1, -1, 1, -1]


# ---------------------------------------------------------------- BN affine
def _round_f32(fr):
    """Exact round-to-nearest-even of a Fraction to float32."""
    c = np.float32(float(fr))
    cands = {c, np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(-np.inf))}
    best = None
    for t in cands:
        d = abs(Fraction(float(t)) - fr)
        even = (int(np.float32(t).view(np.uint32)) & 1) == 0
        key = (d, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, t)
    return best[1]


def test_bn_affine_is_one_fused_rounding(oracle):
    g = rng(11)
    x = g.standard_normal((2, 3, 4, 5)).astype(np.float32)
    scale = (1.0 + 0.3 * g.standard_normal(3)).astype(np.float32)
    shift = (0.2 * g.standard_normal(3)).astype(np.float32)
    y = oracle.bn_affine(x, scale, shift)
    differs_from_two_roundings = 0
    for n, c, h, w in itertools.product(range(2), range(3), range(4), range(5)):
        exact = Fraction(float(scale[c])) * Fraction(float(x[n, c, h, w])) + Fraction(float(shift[c]))
        assert y[n, c, h, w] == _round_f32(exact)
        two = np.float32(np.float32(scale[c] * x[n, c, h, w]) + shift[c])
        differs_from_two_roundings += int(two != y[n, c, h, w])
    assert differs_from_two_roundings > 0      # the test can tell fma from mul+add
    assert np.array_equal(oracle.bn_affine(x, None, None), x)


# ---------------------------------------------------------------- A and K
def test_A_is_channel_mean_of_abs(oracle):
    y = rng(21).standard_normal((3, 7, 4, 6)).astype(np.float32)
    A = oracle.channel_abs_mean(y)
    assert A.shape == (3, 4, 6)
    exact = np.abs(y.astype(np.float64)).mean(axis=1)
    assert np.allclose(A, exact, rtol=1e-7, atol=0)
    # constant magnitude -> A is that constant, whatever the signs
    s = np.where(rng(22).random((2, 5, 3, 3)) < 0.5, -0.25, 0.25).astype(np.float32)
    assert np.array_equal(oracle.channel_abs_mean(s), np.full((2, 3, 3), 0.25, np.float32))


@pytest.mark.parametrize("kh,kw,stride,pad", [(3, 3, 1, 1), (5, 5, 1, 2), (3, 3, 2, 1),
                                               (2, 4, 1, 1), (7, 7, 1, 3), (1, 1, 2, 0)])
def test_K_matches_library_box_filter(oracle, kh, kw, stride, pad):
    """K = A * k, k_ij = 1/(w h), zero padded (Section 3.2): the same thing as an
    average pool that counts padded cells (library routine, fp64)."""
    A = np.abs(rng(31).standard_normal((2, 9, 11))).astype(np.float32)
    K = oracle.box_filter(A, kh, kw, stride, pad)
    ref = F.avg_pool2d(torch.from_numpy(A).double()[:, None], (kh, kw), stride, pad,
                       count_include_pad=True)[:, 0].numpy()
    assert K.shape == ref.shape
    assert np.allclose(K, ref, rtol=1e-6, atol=0)


def test_K_special_cases(oracle):
    A = np.abs(rng(32).standard_normal((2, 6, 5))).astype(np.float32)
    assert np.array_equal(oracle.box_filter(A, 1, 1, 1, 0), A)          # 1x1 filter: K = A
    # "full" convolution (pad = k-1, stride 1): every A value is counted kh*kw times
    K = oracle.box_filter(A, 3, 3, 1, 2)
    assert np.isclose(K.astype(np.float64).sum(), A.astype(np.float64).sum(), rtol=1e-6)
    # constant A: interior K equals the constant, corners see (k+1)/2 squared cells
    c = np.full((1, 8, 8), 0.5, np.float32)
    K = oracle.box_filter(c, 3, 3, 1, 1)
    assert np.all(K[0, 1:-1, 1:-1] == 0.5)
    assert np.isclose(K[0, 0, 0], 0.5 * 4 / 9) and np.isclose(K[0, 0, 3], 0.5 * 6 / 9)


# ---------------------------------------------------------------- binary dot / conv
def _pack(bits):
    """Test-only packing: list of +-1 -> python int, bit i set for +1."""
    v = 0
    for i, b in enumerate(bits):
        if b > 0:
            v |= 1 << i
    return v


@pytest.mark.parametrize("n", [1, 31, 32, 33, 96, 100])
def test_xnor_popcount_identity(oracle, n):
    """Section 3.2: a dot product of +-1 vectors is XNOR + bitcount:
    a.b = n - 2 popcount(bits(a) xor bits(b)).  1x1 'images' make the oracle's
    convolution a plain dot product."""
    g = rng(40 + n)
    a = np.where(g.random((4, n)) < 0.5, -1, 1).astype(np.int8)
    b = np.where(g.random((3, n)) < 0.5, -1, 1).astype(np.int8)
    acc = oracle.binconv_acc(a.reshape(4, n, 1, 1), b.reshape(3, n, 1, 1), 1, 0)
    for i in range(4):
        for j in range(3):
            x = _pack(a[i]) ^ _pack(b[j])
            assert acc[i, j, 0, 0] == n - 2 * bin(x).count("1")


CONV_CASES = [
    # N, C, H, W, Co, kh, kw, stride, pad
    (2, 5, 6, 7, 3, 3, 3, 1, 1),
    (1, 33, 5, 4, 2, 3, 2, 1, 1),
    (2, 4, 9, 8, 3, 5, 5, 1, 2),
    (2, 6, 9, 10, 4, 3, 3, 2, 1),
    (1, 3, 7, 7, 2, 7, 7, 1, 3),
    (2, 8, 5, 6, 3, 1, 1, 1, 0),
    (1, 4, 6, 6, 2, 3, 3, 1, 0),
    (1, 4, 8, 9, 2, 1, 1, 2, 0),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_binconv_acc_matches_library_conv_of_signs(oracle, case):
    """sign(I) (*) sign(W) with 'padded taps add 0' is the zero-padded dense
    convolution of the two +-1 tensors: exact in fp64 (library routine)."""
    N, C, H, W, Co, kh, kw, s, p = case
    g = rng(sum(case))
    Hs = np.where(g.random((N, C, H, W)) < 0.5, -1, 1).astype(np.int8)
    B = np.where(g.random((Co, C, kh, kw)) < 0.5, -1, 1).astype(np.int8)
    acc = oracle.binconv_acc(Hs, B, s, p)
    ref = F.conv2d(torch.from_numpy(Hs).double(), torch.from_numpy(B).double(),
                   stride=s, padding=p).numpy()
    assert acc.shape == ref.shape
    assert np.array_equal(acc.astype(np.float64), ref)


def _valid_taps(H, W, kh, kw, s, p):
    ones = torch.ones(1, 1, H, W, dtype=torch.float64)
    return F.conv2d(ones, torch.ones(1, 1, kh, kw, dtype=torch.float64), stride=s, padding=p)[0, 0].numpy()


@pytest.mark.parametrize("case", CONV_CASES)
def test_acc_invariants(oracle, case):
    """|acc| <= valid taps * C, same parity as it; equality when the window
    equals the filter."""
    N, C, H, W, Co, kh, kw, s, p = case
    g = rng(1 + sum(case))
    Hs = np.where(g.random((N, C, H, W)) < 0.5, -1, 1).astype(np.int8)
    B = np.where(g.random((Co, C, kh, kw)) < 0.5, -1, 1).astype(np.int8)
    acc = oracle.binconv_acc(Hs, B, s, p)
    nv = (_valid_taps(H, W, kh, kw, s, p) * C).astype(np.int64)
    assert np.all(np.abs(acc) <= nv[None, None])
    assert np.all((acc - nv[None, None]) % 2 == 0)
    # all-(+1) input against all-(+1) filter: acc = number of valid taps * C
    acc1 = oracle.binconv_acc(np.ones((1, C, H, W), np.int8), np.ones((1, C, kh, kw), np.int8), s, p)
    assert np.array_equal(acc1[0, 0], nv)
    # flipping every weight flips every accumulator
    assert np.array_equal(oracle.binconv_acc(Hs, -B, s, p), -acc)


@pytest.mark.parametrize("case", CONV_CASES)
def test_block_is_exact_dense_conv_for_constant_magnitudes(oracle, case):
    """Eq. 10: gamma* = beta* alpha* holds with equality when |X_i| and |W_i|
    are constant, so for x in {+-c1}, w in {+-c2} the block must reproduce the
    dense convolution exactly wherever the window is fully inside the image,
    and dense * valid_taps/(kh kw) at the zero-padded border (K divides by the
    full kh*kw)."""
    N, C, H, W, Co, kh, kw, s, p = case
    g = rng(2 + sum(case))
    c1, c2 = 0.5, 0.125
    x = np.where(g.random((N, C, H, W)) < 0.5, -c1, c1).astype(np.float32)
    w = np.where(g.random((Co, C, kh, kw)) < 0.5, -c2, c2).astype(np.float32)
    r = oracle.xnor_block(x, w, s, p)
    dense = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(),
                     stride=s, padding=p).numpy()
    frac = _valid_taps(H, W, kh, kw, s, p) / (kh * kw)
    expect = dense * frac[None, None]
    assert np.allclose(r.out, expect, rtol=1e-6, atol=0)
    inner = frac == 1.0
    if inner.any():
        assert np.allclose(r.out[:, :, inner], dense[:, :, inner], rtol=1e-6, atol=0)
    assert np.all(r.alpha == np.float32(c2)) and np.all(r.A == np.float32(c1))


def test_block_composition_on_gaussian_data(oracle):
    """Eq. 11 assembled from independently pinned pieces: library conv of the
    signs, library box filter of mean|y|, per-filter mean|W|, and the BN
    affine in front of BOTH sign and A."""
    g = rng(77)
    N, C, H, W, Co, kh, kw, s, p = 2, 6, 7, 8, 4, 3, 3, 1, 1
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, kh, kw)).astype(np.float32)
    scale = (1 + 0.5 * g.standard_normal(C)).astype(np.float32)
    shift = g.standard_normal(C).astype(np.float32)
    res = g.standard_normal((N, Co, H, W)).astype(np.float32)
    r = oracle.xnor_block(x, w, s, p, scale, shift, res)
    y = torch.from_numpy(x).double() * torch.from_numpy(scale).double()[None, :, None, None] \
        + torch.from_numpy(shift).double()[None, :, None, None]
    sg = torch.where(y >= 0, 1.0, -1.0).double()
    sw = torch.where(torch.from_numpy(w) >= 0, 1.0, -1.0).double()
    acc = F.conv2d(sg, sw, stride=s, padding=p)
    A = y.abs().mean(dim=1, keepdim=True)
    K = F.avg_pool2d(A, (kh, kw), s, p, count_include_pad=True)
    alpha = torch.from_numpy(w).double().abs().mean(dim=(1, 2, 3))
    out = acc * K * alpha[None, :, None, None] + torch.from_numpy(res).double()
    assert np.array_equal(r.acc, acc.numpy().astype(np.int32))
    assert np.allclose(r.out, out.numpy(), rtol=2e-6, atol=2e-6)
    assert np.allclose(r.K, K[:, 0].numpy(), rtol=1e-6)


def test_structure_of_the_scaling(oracle):
    """K is shared by all filters and is per image; alpha is per filter
    (Section 3.1 and Eq. 11)."""
    g = rng(88)
    x = g.standard_normal((2, 5, 6, 6)).astype(np.float32)
    w = g.standard_normal((3, 5, 3, 3)).astype(np.float32)
    w[1] = np.abs(w[1]) * np.sign(w[0]) * 0.3 + np.where(w[0] >= 0, 1e-3, -1e-3)  # same signs as filter 0
    r = oracle.xnor_block(x, w, 1, 1)
    assert np.array_equal(r.acc[:, 0], r.acc[:, 1])
    assert np.allclose(r.out[:, 0] / r.alpha[0], r.out[:, 1] / r.alpha[1], rtol=1e-5, atol=1e-6)
    # scaling one filter by t>0 scales its outputs by t, accumulators unchanged
    w2 = w.copy(); w2[2] *= 4.0
    r2 = oracle.xnor_block(x, w2, 1, 1)
    assert np.array_equal(r2.acc, r.acc)
    assert np.array_equal(r2.out[:, 2], 4.0 * r.out[:, 2]) and np.array_equal(r2.out[:, :2], r.out[:, :2])
    # scaling one image by t>0 scales that image's outputs only
    x2 = x.copy(); x2[1] *= 2.0
    r3 = oracle.xnor_block(x2, w, 1, 1)
    assert np.array_equal(r3.out[1], 2.0 * r.out[1]) and np.array_equal(r3.out[0], r.out[0])


def test_shortcut_conv_matches_library(oracle):
    g = rng(99)
    x = g.standard_normal((2, 6, 8, 9)).astype(np.float32)
    w = g.standard_normal((5, 6, 1, 1)).astype(np.float32)
    for stride in (1, 2):
        out = oracle.shortcut_conv1x1(x, w, stride)
        ref = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), stride=stride).numpy()
        assert out.shape == ref.shape
        assert np.allclose(out, ref, rtol=1e-6, atol=1e-6)


# ---------------------------------------------------------------- Section 4.1
# ---------------------------------------------------------------- Pool (Section 3.2, block B-A-C-P)
@pytest.mark.parametrize("case", [(2, 3, 9, 7, 3, 2, 0), (1, 4, 8, 11, 3, 2, 1), (2, 2, 6, 6, 2, 2, 0),
                                  (1, 1, 5, 4, 5, 1, 2), (3, 2, 7, 7, 3, 1, 1)])
def test_maxpool_matches_library_routine(oracle, case):
    """torch's max_pool2d (fp64, floor mode, -inf padding) is an independent statement of the
    same definition; maxima of fp32 values are exact, so the match is bit for bit."""
    N, C, H, W, k, s, p = case
    x = rng(sum(case)).standard_normal((N, C, H, W)).astype(np.float32)
    want = F.max_pool2d(torch.from_numpy(x).double(), k, s, p).numpy()
    assert np.array_equal(oracle.maxpool2d(x, k, s, p).astype(np.float64), want)
    want_relu = F.max_pool2d(torch.relu(torch.from_numpy(x).double()), k, s, p).numpy()
    assert np.array_equal(oracle.maxpool2d(x, k, s, p, relu=True).astype(np.float64), want_relu)


def test_maxpool_special_cases(oracle):
    g = rng(123)
    x = g.standard_normal((2, 3, 6, 5)).astype(np.float32)
    # a 1 x 1 window at stride 1 is the identity; with ReLU it is max(x, 0)
    assert np.array_equal(oracle.maxpool2d(x, 1, 1), x)
    assert np.array_equal(oracle.maxpool2d(x, 1, 1, relu=True), np.maximum(x, 0.0))
    # ReLU commutes with the maximum (both are monotone)
    assert np.array_equal(oracle.maxpool2d(x, 3, 2, 1, relu=True),
                          np.maximum(oracle.maxpool2d(x, 3, 2, 1), 0.0))
    # a window that covers the whole plane returns the plane's maximum, padding never wins
    neg = -np.abs(x) - 1.0
    full = oracle.maxpool2d(neg, 6, 6, 1)[:, :, 0, 0]
    assert np.array_equal(full, neg[:, :, :5, :5].max(axis=(2, 3)))
    # brute force over windows, written with slices only
    k, s = 2, 2
    got = oracle.maxpool2d(x, k, s)
    for oy in range(got.shape[2]):
        for ox in range(got.shape[3]):
            assert np.array_equal(got[:, :, oy, ox],
                                  x[:, :, oy * s:oy * s + k, ox * s:ox * s + k].max(axis=(2, 3)))


def test_speedup_model_reproduces_printed_value(oracle):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "efficiency_model.txt"))
            if l.strip() and not l.startswith("#")]
    assert rows
    for c, n_w, printed, nd in rows:
        assert round(oracle.speedup_model(float(c), float(n_w)), int(nd)) == float(printed)
    # first-layer-like shape (c=3, 1x1): "not considerably high"
    assert oracle.speedup_model(3, 1) < 3.0
    # the model's limit for large c*N_W is the word width
    assert 63.9 < oracle.speedup_model(1e9, 9) < 64.0
