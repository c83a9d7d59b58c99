"""Binary-Weight-Network convolution (Section 3.1, Eq. 1) on the GPU against the oracle.

The GPU rounds the (normalised) inputs to bfloat16 once and adds/subtracts them in fp32 on the
tensor cores; the oracle rounds the same values with its own bfloat16 routine and sums in fp64.
Products are exact on both sides, so the only difference is the fp32 accumulation over
n = C_in*k_h*k_w terms; measured, it stays below 3e-7 of the largest output magnitude, so the
tolerance is the one every fp32 comparison here uses (REL_TOL = 1e-5)."""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from paper_1603_05279_b200 import workloads as wl
from util import REL_TOL, GuardSet, assert_close, dev, host

pytestmark = pytest.mark.gpu


def bwn_tol(C, kh, kw):
    return REL_TOL


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def run_bwn(x, w, stride, pad, scale=None, shift=None, residual=None, flags=0, alias=False):
    N, C, H, W = x.shape
    Co, _, kh, kw = w.shape
    d = X.make_desc(N, C, H, W, Co, kh, kw, stride, pad, flags)
    gs = GuardSet()
    wp, alpha = X.alloc_weights(Co, C, kh, kw)
    xs = gs.new("x_stream", (X.xnor_bwn_input_elems(d),), torch.bfloat16)
    out = gs.like("out", X.alloc_out(d))
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_bwn_prepare_input(dev(x), None if scale is None else dev(scale),
                             None if shift is None else dev(shift), d, xs)
    res = None
    if residual is not None:
        if alias:
            out.copy_(dev(residual))
            res = out
        else:
            res = dev(residual)
    X.xnor_bwn_conv2d_forward(xs, wp, alpha, res, d, out)
    X.xnor_check_device()
    gs.check()
    return host(out), host(alpha), xs


def oracle_bwn(oracle, x, w, stride, pad, scale=None, shift=None, residual=None, relu=False):
    y = oracle.bn_affine(x, scale, shift) if scale is not None else x
    Bm, alpha = oracle.binarize_weights(w)
    out = oracle.bwn_conv(oracle.round_bf16(y), Bm, alpha, stride, pad, residual)
    return oracle.relu(out) if relu else out


SHAPES = [
    # N, C, H, W, Co, kh, kw, stride, pad
    (1, 64, 14, 14, 64, 3, 3, 1, 1),
    (2, 3, 9, 11, 5, 3, 3, 1, 1),         # fewer than 16 channels
    (3, 96, 13, 13, 70, 5, 5, 1, 2),
    (2, 100, 7, 7, 33, 3, 3, 1, 1),       # channel tail inside a 16-channel step
    (2, 64, 17, 15, 64, 3, 3, 2, 1),      # stride 2
    (2, 32, 14, 14, 64, 1, 1, 1, 0),
    (1, 40, 14, 14, 16, 7, 7, 1, 3),
    (2, 64, 8, 8, 32, 3, 3, 1, 0),
    (1, 64, 6, 9, 8, 3, 2, 1, 1),         # rectangular filter
    (2, 33, 10, 10, 9, 3, 3, 2, 0),
    (1, 8, 1, 1, 4, 1, 1, 1, 0),          # one pixel
    (1, 288, 9, 9, 130, 3, 3, 1, 1),      # two filter slabs
    (5, 200, 14, 14, 272, 3, 3, 1, 1),    # three slabs, several tiles
]


@pytest.mark.parametrize("shape", SHAPES)
def test_bwn_parity(oracle, shape):
    N, C, H, W, Co, kh, kw, s, p = shape
    g = rng(sum(shape) + 1)
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, kh, kw)).astype(np.float32)
    out, alpha, _ = run_bwn(x, w, s, p)
    assert_close(alpha, oracle.binarize_weights(w)[1], "alpha")
    assert_close(out, oracle_bwn(oracle, x, w, s, p), "out", rel=bwn_tol(C, kh, kw))


def test_bwn_with_bn_residual_and_relu(oracle):
    g = rng(5)
    N, C, H, W, Co = 3, 70, 13, 13, 40
    x = (2.0 + 3.0 * g.standard_normal((N, C, H, W))).astype(np.float32)
    w = (0.05 * g.standard_normal((Co, C, 3, 3))).astype(np.float32)
    scale = (1.0 / 3.0 + 0.05 * g.standard_normal(C)).astype(np.float32)
    shift = (-2.0 / 3.0 + 0.05 * g.standard_normal(C)).astype(np.float32)
    res = g.standard_normal((N, Co, H, W)).astype(np.float32)
    tol = bwn_tol(C, 3, 3)
    want = oracle_bwn(oracle, x, w, 1, 1, scale, shift, res)
    assert_close(run_bwn(x, w, 1, 1, scale, shift, res)[0], want, "out", rel=tol)
    assert_close(run_bwn(x, w, 1, 1, scale, shift, res, alias=True)[0], want, "out (residual = out)", rel=tol)
    got = run_bwn(x, w, 1, 1, scale, shift, res, flags=B.XNOR_FLAG_RELU)[0]
    assert_close(got, oracle.relu(want), "out with ReLU", rel=tol)
    assert got.min() >= 0.0


def test_bwn_input_is_the_rounded_stream(oracle):
    """The prepared stream holds exactly the oracle's bfloat16 values of the (normalised) input
    and zeros elsewhere: as a multiset per channel, whatever the private layout is."""
    g = rng(6)
    N, C, H, W = 2, 20, 6, 7
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((4, C, 3, 3)).astype(np.float32)
    _, _, xs = run_bwn(x, w, 1, 1)
    got = np.sort(host(xs.float()).ravel())
    want = np.sort(oracle.round_bf16(x).ravel())
    nz = got[got != 0.0]
    assert np.array_equal(nz, want[want != 0.0])


def test_bwn_constant_magnitude_weights_give_the_dense_convolution(oracle):
    """Eq. 1 with equality: w in {+-c} and inputs representable in bfloat16 -> the dense
    zero-padded convolution, exactly where the fp32 sums are exact (small integers)."""
    import torch.nn.functional as F
    g = rng(8)
    x = g.integers(-4, 5, (2, 64, 10, 10)).astype(np.float32)
    w = np.where(g.random((16, 64, 3, 3)) < 0.5, -0.25, 0.25).astype(np.float32)
    out, _, _ = run_bwn(x, w, 1, 1)
    dense = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), padding=1).numpy()
    assert np.array_equal(out.astype(np.float64), dense)


@pytest.mark.parametrize("li", range(len(wl.RESNET18)))
def test_bwn_resnet_layers_at_full_batch(oracle, li):
    s = wl.RESNET18[li]
    x = wl.make_input(s, wl.layer_seed("resnet18", li))
    w = wl.make_weights(s, wl.layer_seed("resnet18", li))
    d = X.desc_of(s)
    wp, alpha = X.alloc_weights(s.C_out, s.C_in, s.k, s.k)
    xs = X.alloc_bwn_input(d)
    out = X.alloc_out(d)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_bwn_prepare_input(dev(x), None, None, d, xs)
    X.xnor_bwn_conv2d_forward(xs, wp, alpha, None, d, out)
    X.xnor_check_device()
    for n in (0, s.N // 2, s.N - 1):
        want = oracle_bwn(oracle, x[n:n + 1], w, s.stride, s.pad)
        assert_close(host(out[n:n + 1]), want, "%s image %d" % (s.name, n), rel=bwn_tol(s.C_in, s.k, s.k))


def test_bwn_reports_what_it_does_not_cover():
    d = X.make_desc(1, 16, 12, 12, 12, 3, 3, 3, 1)       # stride 3
    with pytest.raises(X.XnorError) as e:
        X.xnor_bwn_prepare_input(torch.empty((1, 16, 12, 12), device="cuda"), None, None, d,
                                 torch.empty(4096, dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == B.XNOR_ERR_UNSUPPORTED
    wide = X.make_desc(1, 16, 8, 200, 16, 3, 3, 1, 1)    # a tile's window exceeds 256 positions
    assert X.xnor_bwn_input_elems(wide) > 0
    with pytest.raises(X.XnorError) as e:
        X.xnor_bwn_conv2d_forward(torch.empty(8, dtype=torch.bfloat16, device="cuda"),
                                  *X.alloc_weights(16, 16, 3, 3), None, wide, X.alloc_out(wide))
    assert e.value.status == B.XNOR_ERR_UNSUPPORTED
