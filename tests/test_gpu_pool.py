"""GPU parity of the Pool layer (max pooling, optional ReLU) against the CPU oracle.
A maximum of fp32 values is exact, so the results must be identical."""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from util import dev, host

pytestmark = pytest.mark.gpu

# (N, C, H, W, k, stride, pad): AlexNet's 3x3/2 pools on the conv2 and conv5 outputs; ResNet's
# 3x3/2 pad 1; odd sizes; a 1x1 window; a window as large as the plane; planes beyond the
# shared-memory path (120 x 100 floats)
CASES = [(4, 256, 27, 27, 3, 2, 0), (3, 256, 13, 13, 3, 2, 0), (2, 64, 56, 56, 3, 2, 1),
         (2, 5, 9, 7, 2, 2, 0), (1, 3, 8, 11, 3, 1, 1), (2, 2, 5, 4, 1, 1, 0), (2, 3, 6, 6, 6, 6, 1),
         (1, 2, 120, 100, 3, 2, 1), (1, 1, 1, 1, 1, 1, 0), (3, 70, 13, 13, 5, 3, 2)]


@pytest.mark.parametrize("relu", [False, True])
@pytest.mark.parametrize("case", CASES)
def test_maxpool_parity(oracle, case, relu):
    N, C, H, W, k, s, p = case
    x = np.random.Generator(np.random.Philox(sum(case))).standard_normal((N, C, H, W)).astype(np.float32)
    want = oracle.maxpool2d(x, k, s, p, relu=relu)
    out = torch.empty(want.shape, dtype=torch.float32, device="cuda")
    X.xnor_maxpool2d(dev(x), k, s, p, relu, out)
    torch.cuda.synchronize()
    assert np.array_equal(host(out), want)


def test_maxpool_after_binconv_closes_the_block(oracle):
    """B-A-C-P on one small layer: the pooled BinConv output equals the oracle's pooled output
    when both pool the same fp32 tensor (the GPU's), and pooling commutes with the tolerance of
    the block (a maximum does not amplify errors)."""
    g = np.random.Generator(np.random.Philox(31))
    x = g.standard_normal((2, 96, 27, 27)).astype(np.float32)
    w = (0.01 * g.standard_normal((64, 96, 5, 5))).astype(np.float32)
    d = B.xnor_conv_desc(2, 96, 27, 27, 64, 5, 5, 1, 2)
    wp, alpha = X.alloc_weights(64, 96, 5, 5)
    xp, A, K = X.alloc_binactiv(d)
    out = X.alloc_out(d)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
    X.xnor_conv2d_forward(xp, wp, alpha, K, None, d, out, None)
    pooled = torch.empty((2, 64, 13, 13), dtype=torch.float32, device="cuda")
    X.xnor_maxpool2d(out, 3, 2, 0, True, pooled)
    X.xnor_check_device()
    assert np.array_equal(host(pooled), oracle.maxpool2d(host(out), 3, 2, 0, relu=True))
    ref = oracle.maxpool2d(oracle.xnor_block(x, w, 1, 2).out, 3, 2, 0, relu=True)
    assert np.abs(host(pooled) - ref).max() <= 1e-5 * np.abs(ref).max()


def test_maxpool_arguments():
    x = torch.zeros((1, 1, 4, 4), device="cuda")
    out = torch.zeros((1, 1, 2, 2), device="cuda")
    for k, s, p in [(0, 1, 0), (3, 0, 0), (3, 1, 3), (3, 1, -1), (7, 1, 1)]:
        with pytest.raises(X.XnorError) as e:
            X.xnor_maxpool2d(x, k, s, p, False, out)
        assert e.value.status == B.XNOR_ERR_INVALID_ARG
