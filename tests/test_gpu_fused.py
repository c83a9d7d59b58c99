"""BinConv with the next layer's BinActiv fused into its epilogue, against the CPU oracle.

The fused call must produce the fp32 tensor of the plain call bit for bit; the oracle then
applies the next BatchNorm affine, sign and channel mean to THAT tensor (the sign of a value
near zero depends on its last bit, so both sides must start from the same fp32 values), and the
packed bits must match exactly, A and K within the tolerance."""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from util import GuardSet, assert_close, dev, host, unpack_activations

pytestmark = pytest.mark.gpu

ENGINES = [B.XNOR_ENGINE_AUTO, B.XNOR_ENGINE_UMMA_SINGLE, B.XNOR_ENGINE_UMMA_STREAM,
           B.XNOR_ENGINE_UMMA_PAIR, B.XNOR_ENGINE_UMMA_PAIR_STREAM]
# (N, C, H, W, Co, k, stride, pad, next k, next stride, next pad, residual)
CASES = [(3, 64, 20, 20, 64, 3, 1, 1, 3, 1, 1, True),       # one slab of 64: two pairs of groups
         (2, 96, 13, 13, 384, 3, 1, 1, 3, 1, 1, False),     # three slabs
         (2, 64, 18, 18, 128, 3, 2, 1, 3, 1, 1, False),     # stride 2
         (2, 40, 9, 11, 32, 5, 1, 2, 1, 1, 0, True),        # one pair only; channel tail in the input
         (4, 128, 14, 14, 256, 3, 1, 1, 3, 2, 1, True),
         (2, 64, 10, 10, 512, 3, 2, 1, 3, 1, 1, False),     # slabs of 192: the last one holds 128 filters
         (1, 32, 7, 7, 288, 1, 1, 0, 3, 1, 1, True)]


def _run(case, engine, with_out, with_bn):
    N, C, H, W, Co, k, s, p, k2, s2, p2, use_res = case
    g = np.random.Generator(np.random.Philox(sum(case[:8]) + 7))
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, k, k)).astype(np.float32)
    d = B.xnor_conv_desc(N, C, H, W, Co, k, k, s, p)
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    d2 = B.xnor_conv_desc(N, Co, Ho, Wo, 32, k2, k2, s2, p2)
    res = dev(g.standard_normal((N, Co, Ho, Wo)).astype(np.float32)) if use_res else None
    scale = (0.5 + g.random(Co)).astype(np.float32) if with_bn else None
    shift = (0.3 * g.standard_normal(Co)).astype(np.float32) if with_bn else None
    wp, alpha = X.alloc_weights(Co, C, k, k)
    xp, A, K = X.alloc_binactiv(d)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
    X.xnor_set_engine(engine)
    try:
        out_ref = X.alloc_out(d)
        X.xnor_conv2d_forward(xp, wp, alpha, K, res, d, out_ref, None)
        parts = X.xnor_conv2d_binactiv_parts(d)
        assert parts >= 1, (case, engine)
        gs = GuardSet()
        xp2, A2, K2 = (gs.like(n, t) for n, t in zip(("x_packed_next", "A", "K"), X.alloc_binactiv(d2)))
        A_parts = gs.new("A_parts", (parts, N, Ho, Wo))
        out = gs.like("out", X.alloc_out(d)) if with_out else None
        X.xnor_conv2d_forward_binactiv(xp, wp, alpha, K, res, d, out,
                                       dev(scale) if with_bn else None, dev(shift) if with_bn else None,
                                       xp2, A_parts)
        X.xnor_binactiv_finish(A_parts, parts, d2, A2, K2)
    finally:
        X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
    X.xnor_check_device()
    gs.check()
    return out_ref, out, xp2, A2, K2, scale, shift, (k2, s2, p2)


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("case", CASES)
def test_fused_binactiv_parity(oracle, case, engine):
    Co = case[4]
    for with_out, with_bn in [(True, True), (False, False)]:
        out_ref, out, xp2, A2, K2, scale, shift, (k2, s2, p2) = _run(case, engine, with_out, with_bn)
        if with_out:
            assert torch.equal(out, out_ref)
        o = host(out_ref)
        sc = scale if with_bn else np.ones(Co, np.float32)
        sh = shift if with_bn else np.zeros(Co, np.float32)
        y = oracle.bn_affine(o, sc, sh)
        assert np.array_equal(unpack_activations(host(xp2), Co), oracle.sign(y).reshape(y.shape))
        A_or = oracle.channel_abs_mean(y)
        assert_close(host(A2), A_or, "A of the fused BinActiv")
        assert_close(host(K2), oracle.box_filter(A_or, k2, k2, s2, p2), "K of the fused BinActiv")


def test_fused_call_reports_what_it_does_not_cover():
    d = B.xnor_conv_desc(1, 32, 8, 8, 40, 3, 3, 1, 1)        # C_out not a multiple of 32
    assert X.xnor_conv2d_binactiv_parts(d) == 0
    X.xnor_set_engine(B.XNOR_ENGINE_POPC)
    try:
        assert X.xnor_conv2d_binactiv_parts(B.xnor_conv_desc(1, 32, 8, 8, 64, 3, 3, 1, 1)) == 0
    finally:
        X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
