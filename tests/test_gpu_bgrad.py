"""Backward convolution with a binarised gradient (Section 3.2, "Binary Gradient") on the GPU
against the oracle.

gmax is a maximum (exact) and the transposed sign words are bits (exact); the result is a sum of
+-bf16(gmax * alpha[co]) terms, the products rounded identically on both sides (fp32 product,
bfloat16 round to nearest even), accumulated in fp32 on the GPU and in fp64 by the oracle: within
REL_TOL of the largest magnitude, like every fp32 comparison here."""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from util import GuardSet, assert_close, dev, host, unpack_weights

pytestmark = pytest.mark.gpu


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def run_backward(grad, w, d):
    Co, C, kh, kw = w.shape
    gs = GuardSet()
    wp, alpha = X.alloc_weights(Co, C, kh, kw)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    wT = gs.like("wT_packed", X.alloc_weights_transposed(Co, C, kh, kw))
    X.xnor_binarize_weights_transposed(dev(w), wT)
    gmax0, stream0, gin0 = X.alloc_bgrad(d)
    gmax, stream, gin = gs.like("gmax", gmax0), gs.like("g_stream", stream0), gs.like("grad_in", gin0)
    gmax.fill_(123.0); gin.fill_(float("nan"))
    X.xnor_binary_gradient_backward(dev(grad), wT, alpha, d, gmax, stream, gin)
    X.xnor_check_device()
    gs.check()
    return host(wT), host(alpha), host(gmax), host(gin)


# N, C, H, W, Co, k, pad
SHAPES = [(2, 64, 14, 14, 64, 3, 1), (3, 70, 9, 11, 40, 5, 2), (2, 32, 8, 8, 16, 1, 0),
          (5, 96, 13, 12, 130, 3, 0), (2, 48, 20, 17, 33, 3, 2), (130, 16, 7, 7, 24, 3, 1),
          (4, 256, 13, 13, 384, 3, 1)]


@pytest.mark.parametrize("shape", SHAPES)
def test_binary_gradient_backward_parity(oracle, shape):
    N, C, H, W, Co, k, p = shape
    g = rng(sum(shape) + 5)
    w = g.standard_normal((Co, C, k, k)).astype(np.float32)
    Ho, Wo = H + 2 * p - k + 1, W + 2 * p - k + 1
    grad = (g.standard_normal((N, Co, Ho, Wo)) * g.uniform(0.01, 3.0, (N, 1, 1, 1))).astype(np.float32)
    grad[0, 0, 0, :2] = [0.0, -0.0]                        # sign(0) = +1 for both zeros
    d = X.make_desc(N, C, H, W, Co, k, k, 1, p)
    wT, alpha, gmax, gin = run_backward(grad, w, d)
    Bm, alpha_or = oracle.binarize_weights(w)
    # the transposed words: filter c of the backward convolution, channels co, taps turned
    assert np.array_equal(unpack_weights(wT, Co, k, k), Bm.transpose(1, 0, 2, 3)[:, :, ::-1, ::-1])
    gmax_or, gin_or = oracle.binary_gradient_backward(grad, Bm, alpha, p, (H, W), round_products=True)
    assert_close(alpha, alpha_or, "alpha")
    assert np.array_equal(gmax, gmax_or)
    assert_close(gin, gin_or, "grad_in")
    assert np.isfinite(gin).all()


def test_binary_gradient_backward_at_benchmark_batch(oracle):
    """AlexNet conv3's backward convolution at batch 256, the oracle on three images."""
    N, C, H, W, Co, k, p = 256, 256, 13, 13, 384, 3, 1
    g = rng(77)
    w = (0.01 * g.standard_normal((Co, C, k, k))).astype(np.float32)
    grad = (1e-3 * g.standard_normal((N, Co, H, W))).astype(np.float32)
    d = X.make_desc(N, C, H, W, Co, k, k, 1, p)
    wT, alpha, gmax, gin = run_backward(grad, w, d)
    Bm, _ = oracle.binarize_weights(w)
    assert np.array_equal(gmax, np.abs(grad).reshape(N, -1).max(axis=1))
    for n in (0, 131, 255):
        _, want = oracle.binary_gradient_backward(grad[n:n + 1], Bm, alpha, p, (H, W), round_products=True)
        assert_close(gin[n:n + 1], want, "grad_in of image %d" % n)


def test_binary_gradient_backward_refuses_what_it_does_not_cover():
    d2 = X.make_desc(2, 64, 14, 14, 64, 3, 3, 2, 1)                   # stride 2
    assert X.xnor_bgrad_stream_elems(d2) == 0
    d1 = X.make_desc(2, 64, 14, 14, 64, 3, 3, 1, 1)
    assert X.xnor_bgrad_stream_elems(d1) > 0
    wT = X.alloc_weights_transposed(64, 64, 3, 3)
    gmax, stream, gin = X.alloc_bgrad(d1)
    grad = torch.zeros((2, 64, 7, 7), device="cuda")
    alpha = torch.ones((64,), device="cuda")
    with pytest.raises(X.XnorError) as e:
        X.xnor_binary_gradient_backward(grad, wT, alpha, d2, gmax, stream, gin)
    assert e.value.status == B.XNOR_ERR_UNSUPPORTED
    with pytest.raises(X.XnorError) as e:
        X.xnor_binary_gradient_backward(grad, wT, None, d1, gmax, stream, gin)
    assert e.value.status == B.XNOR_ERR_INVALID_ARG
    # an all-zero gradient has gmax = 0 and gives an all-zero result
    g0 = torch.zeros((2, 64, 14, 14), device="cuda")
    X.xnor_binarize_weights_transposed(torch.ones((64, 64, 3, 3), device="cuda"), wT)
    X.xnor_binary_gradient_backward(g0, wT, alpha, d1, gmax, stream, gin)
    X.xnor_check_device()
    assert float(gmax.abs().max()) == 0.0 and float(gin.abs().max()) == 0.0
