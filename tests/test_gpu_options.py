"""The block's options on the GPU against the oracle: ReLU after BinConv, the border variant of
K (both Section 3.2, "Training XNOR-Networks") and k-bit activations q_k (Section 3.2, "k-bit
Quantization").  Bits, index planes and integer sums identical; fp32 within REL_TOL."""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from util import GuardSet, assert_close, dev, host, unpack_activations

pytestmark = pytest.mark.gpu

ENGINES = [B.XNOR_ENGINE_AUTO, B.XNOR_ENGINE_POPC, B.XNOR_ENGINE_UMMA_STREAM, B.XNOR_ENGINE_UMMA_SINGLE,
           B.XNOR_ENGINE_UMMA_PAIR]
# N, C, H, W, Co, k, stride, pad
SHAPES = [(3, 64, 14, 14, 64, 3, 1, 1), (2, 70, 9, 11, 40, 5, 1, 2), (2, 96, 13, 12, 130, 3, 2, 1),
          (5, 256, 13, 13, 384, 3, 1, 1), (2, 32, 8, 8, 16, 1, 1, 0)]


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def _inputs(shape, seed):
    N, C, H, W, Co, k, s, p = shape
    g = rng(seed)
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, k, k)).astype(np.float32)
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    res = g.standard_normal((N, Co, Ho, Wo)).astype(np.float32)
    scale = (1.0 + 0.2 * g.standard_normal(C)).astype(np.float32)
    shift = (0.2 * g.standard_normal(C)).astype(np.float32)
    return x, w, res, scale, shift


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("shape", SHAPES)
def test_relu_and_valid_taps_flags(oracle, shape, engine):
    N, C, H, W, Co, k, s, p = shape
    x, w, res, scale, shift = _inputs(shape, sum(shape))
    for flags, use_res, with_acc in [(B.XNOR_FLAG_RELU, False, False), (B.XNOR_FLAG_RELU, True, False),
                                     (B.XNOR_FLAG_RELU | B.XNOR_FLAG_K_VALID_TAPS, True, True),
                                     (B.XNOR_FLAG_K_VALID_TAPS, False, False)]:
        d = X.make_desc(N, C, H, W, Co, k, k, s, p, flags)
        gs = GuardSet()
        wp, alpha = X.alloc_weights(Co, C, k, k)
        xp, A, K = (gs.like(n, t) for n, t in zip(("x_packed", "A", "K"), X.alloc_binactiv(d)))
        out = gs.like("out", X.alloc_out(d))
        acc = gs.like("acc", X.alloc_out(d, torch.int32)) if with_acc else None
        X.xnor_binarize_weights(dev(w), wp, alpha)
        X.xnor_binactiv(dev(x), dev(scale), dev(shift), d, xp, A, K)
        X.xnor_set_engine(engine)
        try:
            X.xnor_conv2d_forward(xp, wp, alpha, K, dev(res) if use_res else None, d, out, acc)
        except X.XnorError as e:
            assert engine not in (B.XNOR_ENGINE_AUTO, B.XNOR_ENGINE_POPC) and e.status == B.XNOR_ERR_UNSUPPORTED
            continue
        finally:
            X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
        X.xnor_check_device()
        gs.check()
        r = oracle.xnor_block_ex(x, w, s, p, scale, shift, res if use_res else None,
                                 relu=bool(flags & B.XNOR_FLAG_RELU),
                                 k_valid_taps=bool(flags & B.XNOR_FLAG_K_VALID_TAPS))
        assert_close(host(K), r.K, "K (flags %d)" % flags)
        assert_close(host(out), r.out, "out (flags %d)" % flags)
        if with_acc:
            assert np.array_equal(host(acc), r.acc)
        if flags & B.XNOR_FLAG_RELU:
            assert float(out.min()) >= 0.0 and bool((out == 0).any())


def test_relu_in_the_fused_epilogue(oracle):
    """The fused BinActiv sees the value after ReLU, as the next layer would."""
    N, C, H, W, Co, k = 2, 64, 12, 12, 64, 3
    x, w, res, _, _ = _inputs((N, C, H, W, Co, k, 1, 1), 31)
    g = rng(32)
    nscale = (0.5 + g.random(Co)).astype(np.float32)
    nshift = (-0.4 + 0.1 * g.standard_normal(Co)).astype(np.float32)
    d = X.make_desc(N, C, H, W, Co, k, k, 1, 1, B.XNOR_FLAG_RELU)
    d2 = X.make_desc(N, Co, H, W, 32, 3, 3, 1, 1)
    wp, alpha = X.alloc_weights(Co, C, k, k)
    xp, A, K = X.alloc_binactiv(d)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
    out_ref = X.alloc_out(d)
    X.xnor_conv2d_forward(xp, wp, alpha, K, dev(res), d, out_ref, None)
    parts = X.xnor_conv2d_binactiv_parts(d)
    assert parts >= 1
    xp2, A2, K2 = X.alloc_binactiv(d2)
    A_parts = torch.empty((parts, N, H, W), dtype=torch.float32, device="cuda")
    out = X.alloc_out(d)
    X.xnor_conv2d_forward_binactiv(xp, wp, alpha, K, dev(res), d, out, dev(nscale), dev(nshift), xp2, A_parts)
    X.xnor_binactiv_finish(A_parts, parts, d2, A2, K2)
    X.xnor_check_device()
    assert torch.equal(out, out_ref) and float(out.min()) >= 0.0
    r = oracle.xnor_block_ex(x, w, 1, 1, residual=res, relu=True)
    assert_close(host(out), r.out, "out")
    y = oracle.bn_affine(host(out), nscale, nshift)
    assert np.array_equal(unpack_activations(host(xp2), Co), oracle.sign(y).reshape(y.shape))
    A_or = oracle.channel_abs_mean(y)
    assert_close(host(A2), A_or, "A")
    assert_close(host(K2), oracle.box_filter(A_or, 3, 3, 1, 1), "K")


def test_unknown_flag_bits_are_rejected():
    d = X.make_desc(1, 32, 8, 8, 16, 3, 3, 1, 1, 4)
    with pytest.raises(X.XnorError) as e:
        X.xnor_binactiv(torch.empty((1, 32, 8, 8), device="cuda"), None, None, d, *X.alloc_binactiv(d))
    assert e.value.status == B.XNOR_ERR_INVALID_ARG


def _index_of_planes(planes, C):
    """u32 [k][N][H][W][Cw] bit planes -> index i per value, [N][C][H][W]."""
    idx = 0
    for p in range(planes.shape[0]):
        bits = (unpack_activations(planes[p], C).astype(np.int64) + 1) // 2
        idx = idx + (bits << p)
    return idx


@pytest.mark.parametrize("engine", [B.XNOR_ENGINE_AUTO, B.XNOR_ENGINE_POPC, B.XNOR_ENGINE_UMMA_STREAM])
@pytest.mark.parametrize("kbits", [1, 2, 3])
@pytest.mark.parametrize("shape", [(4, 64, 14, 14, 64, 3, 1, 1), (2, 70, 9, 12, 40, 5, 1, 2),
                                   (4, 96, 13, 12, 130, 3, 2, 1), (4, 256, 13, 13, 384, 3, 1, 1)])
def test_kbit_block_parity(oracle, shape, kbits, engine):
    N, C, H, W, Co, k, s, p = shape
    x, w, res, scale, shift = _inputs(shape, 7 * sum(shape) + kbits)
    x *= 0.6                                   # a good part of the values inside [-1, 1]
    d = X.make_desc(N, C, H, W, Co, k, k, s, p, B.XNOR_FLAG_RELU if kbits == 3 else 0)
    Cw = (C + 31) // 32
    gs = GuardSet()
    wp, alpha = X.alloc_weights(Co, C, k, k)
    planes = gs.new("x_planes", (kbits, N, H, W, Cw), torch.int32)
    _, A0, K0 = X.alloc_binactiv(d)
    A, K = gs.like("A", A0), gs.like("K", K0)
    out = gs.like("out", X.alloc_out(d))
    acc = gs.like("acc", X.alloc_out(d, torch.int32))
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv_kbit(dev(x), dev(scale), dev(shift), d, kbits, planes, A, K)
    X.xnor_set_engine(engine)
    try:
        X.xnor_conv2d_forward_kbit(planes, kbits, wp, alpha, K, dev(res), d, out, acc)
        out_b = torch.empty_like(out)
        X.xnor_conv2d_forward_kbit(planes, kbits, wp, alpha, K, dev(res), d, out_b, None)
    finally:
        X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
    X.xnor_check_device()
    gs.check()
    r = oracle.xnor_block_ex(x, w, s, p, scale, shift, res, kbits=kbits, relu=(kbits == 3))
    m = 2 ** kbits - 1
    assert np.array_equal(2 * _index_of_planes(host(planes), C) - m, r.H.astype(np.int64)), "level codes"
    assert_close(host(A), r.A, "A")
    assert_close(host(K), r.K, "K")
    assert np.array_equal(host(acc), r.acc), "integer sums over level codes"
    assert_close(host(out), r.out, "out")
    assert torch.equal(out, out_b)
    if kbits == 1:
        # one plane = the 1-bit block, bit for bit (A, hence K, is summed in another order by
        # the two BinActiv kernels, so the convolutions are compared on the same K)
        xp, A1, K1 = X.alloc_binactiv(d)
        X.xnor_binactiv(dev(x), dev(scale), dev(shift), d, xp, A1, K1)
        assert_close(host(K1), host(K), "K of the two BinActiv kernels")
        out1 = X.alloc_out(d)
        X.xnor_conv2d_forward(xp, wp, alpha, K, dev(res), d, out1, None)
        assert torch.equal(xp, planes[0]) and torch.equal(out1, out)


def test_kbit_decision_points(oracle):
    """Values on and next to the rounding thresholds of q_k, and outside [-1, 1]."""
    for kbits in (1, 2, 4):
        m = 2 ** kbits - 1
        taus = np.array([(2 * j - 1) / m - 1 for j in range(1, m + 1)], np.float64).astype(np.float32)
        vals = np.concatenate([taus, np.nextafter(taus, np.float32(-2)), np.nextafter(taus, np.float32(2)),
                               np.array([-1.0, 1.0, -1.5, 1.5, 0.0, -0.0, 1e-9, -1e-9], np.float32)])
        C = 32
        n = (len(vals) + C - 1) // C * C
        v = np.resize(vals, n).astype(np.float32)
        x = v.reshape(1, n // C, C, 1).transpose(0, 2, 1, 3).copy()          # [1][C][n/C][1]
        H = x.shape[2]
        d = X.make_desc(1, C, H, 1, 4, 1, 1, 1, 0)
        planes = torch.zeros((kbits, 1, H, 1, 1), dtype=torch.int32, device="cuda")
        _, A, K = X.alloc_binactiv(d)
        X.xnor_binactiv_kbit(dev(x), None, None, d, kbits, planes, A, K)
        torch.cuda.synchronize()
        assert np.array_equal(2 * _index_of_planes(host(planes), C) - m, oracle.quantize_k(x, kbits).astype(np.int64))


@pytest.mark.parametrize("kbits", [1, 2, 3, 7])
@pytest.mark.parametrize("shape", [(160, 96, 27, 27, 5, 2, True), (150, 40, 13, 13, 3, 1, False),
                                   (96, 256, 7, 7, 3, 1, True)])
def test_kbit_binactiv_on_planes_of_odd_size_with_many_images(oracle, shape, kbits):
    """With enough images and planes that are not a multiple of four pixels the k-bit BinActiv is
    one kernel that streams whole images (as for sign bits): level codes identical to the oracle's
    and to the two-kernel path, A and K within tolerance."""
    N, C, H, W, k, p, bn = shape
    g = rng(3 * sum(shape[:6]) + kbits)
    x = (0.6 * g.standard_normal((N, C, H, W))).astype(np.float32)
    scale = (1.0 + 0.2 * g.standard_normal(C)).astype(np.float32) if bn else None
    shift = (0.2 * g.standard_normal(C)).astype(np.float32) if bn else None
    d = X.make_desc(N, C, H, W, 8, k, k, 1, p)
    # one kernel whenever k planes of an image's packed words fit shared memory beside the copies
    assert X.xnor_binactiv_kbit_launches(d, kbits, bn) == (1 if kbits <= 3 else X.xnor_binactiv_kbit_launches(d, kbits, bn))
    Cw = (C + 31) // 32
    gs = GuardSet()
    planes = gs.new("x_planes", (kbits, N, H, W, Cw), torch.int32)
    _, A0, K0 = X.alloc_binactiv(d)
    A, K = gs.like("A", A0), gs.like("K", K0)
    planes.fill_(-1); A.fill_(float("nan")); K.fill_(float("nan"))
    xd = dev(x)
    sc, sh = (None, None) if scale is None else (dev(scale), dev(shift))
    X.xnor_binactiv_kbit(xd, sc, sh, d, kbits, planes, A, K)
    X.xnor_check_device()
    gs.check()
    m = 2 ** kbits - 1
    for n in sorted({0, N // 2, N - 1}):
        y = x[n:n + 1] if scale is None else oracle.bn_affine(x[n:n + 1], scale, shift)
        codes = 2 * _index_of_planes(host(planes[:, n:n + 1]), C) - m
        assert np.array_equal(codes, oracle.quantize_k(y, kbits).astype(np.int64)), n
        A_or = oracle.channel_abs_mean(y)
        assert_close(host(A[n:n + 1]), A_or, "A of image %d" % n)
        assert_close(host(K[n:n + 1]), oracle.box_filter(A_or, k, k, 1, p), "K of image %d" % n)
    # the last images alone take the two-kernel path: same planes
    d8 = X.make_desc(8, C, H, W, 8, k, k, 1, p)
    assert X.xnor_binactiv_kbit_launches(d8, kbits, bn) == 2
    planes8 = torch.empty((kbits, 8, H, W, Cw), dtype=torch.int32, device="cuda")
    _, A8, K8 = X.alloc_binactiv(d8)
    X.xnor_binactiv_kbit(xd[N - 8:].contiguous(), sc, sh, d8, kbits, planes8, A8, K8)
    assert torch.equal(planes8, planes[:, N - 8:])
    assert_close(host(A8), host(A[N - 8:]), "A of the two paths")
