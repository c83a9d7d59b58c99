"""xnor_binactiv_static: BinActiv for callers that cannot allocate device memory.

The ordinary xnor_binactiv wants a caller buffer for the A plane.  A caller that
lives inside a fixed memory plan (or a plug-in that is handed only its inputs
and outputs) has none to give, so this entry point keeps A in a fixed array
inside the library.  These tests call it through the C ABI and compare it with
xnor_binactiv and with the CPU oracle on the same inputs, twice in a row with
different shapes, so that what the first call leaves in the shared array is seen
not to leak into the second; a last case fills the array to its last element.
Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from util import assert_close, dev, host, unpack_activations


def _both(x, scale, shift, d):
    xp_ref, A_ref, K_ref = X.alloc_binactiv(d)
    X.xnor_binactiv(dev(x), dev(scale), dev(shift), d, xp_ref, A_ref, K_ref)
    xp = torch.full_like(xp_ref, -1)
    K = torch.full_like(K_ref, float("nan"))
    B.xnor_binactiv_static(dev(x), dev(scale), dev(shift), d, xp, K)
    torch.cuda.synchronize()
    return host(xp_ref), host(K_ref), host(xp), host(K)


@pytest.mark.gpu
def test_static_scratch_matches_binactiv_on_two_calls_in_a_row(oracle):
    g = np.random.Generator(np.random.Philox(77))
    # first a larger problem, then a smaller one with another geometry: stale A values
    # of the first call lie beyond and between what the second call writes
    for (N, C, H, W, k, s, p) in [(5, 70, 19, 23, 3, 1, 1), (2, 33, 9, 7, 5, 2, 2)]:
        x = g.standard_normal((N, C, H, W)).astype(np.float32)
        scale = (1.0 + 0.1 * g.standard_normal(C)).astype(np.float32)
        shift = (0.1 * g.standard_normal(C)).astype(np.float32)
        d = X.make_desc(N, C, H, W, 8, k, k, s, p)
        xp_ref, K_ref, xp, K = _both(x, scale, shift, d)
        assert np.array_equal(xp, xp_ref), "packed sign bits"
        assert_close(K, K_ref, "K")          # the tolerance every fp32 comparison here uses
        assert np.array_equal(K, K_ref)      # and in fact the same kernels: identical
        # and against the oracle directly, not only through xnor_binactiv
        y = oracle.bn_affine(x, scale, shift)
        assert np.array_equal(unpack_activations(xp, C), oracle.sign(y).reshape(y.shape))
        assert_close(K, oracle.box_filter(oracle.channel_abs_mean(y), k, k, s, p), "K against the oracle")


@pytest.mark.gpu
def test_static_scratch_at_exactly_its_capacity(oracle):
    """N*H*W equal to the array's size: the last element of the array is used, and with this
    many pixels the pack kernel runs in its one-warp-per-pixel-group mode."""
    N, C, H, W = 256, 8, 64, 64
    assert N * H * W == B.BINACTIV_STATIC_MAX_PIXELS
    g = np.random.Generator(np.random.Philox(78))
    x = g.standard_normal((N, C, H, W), dtype=np.float32)
    scale = (1.0 + 0.1 * g.standard_normal(C)).astype(np.float32)
    shift = (0.1 * g.standard_normal(C)).astype(np.float32)
    d = X.make_desc(N, C, H, W, 8, 3, 3, 1, 1)
    xp_ref, K_ref, xp, K = _both(x, scale, shift, d)
    assert np.array_equal(xp, xp_ref) and np.array_equal(K, K_ref)
    for n in (0, N - 1):                       # the last image's A sits at the end of the array
        y = oracle.bn_affine(x[n:n + 1], scale, shift)
        assert np.array_equal(unpack_activations(xp[n:n + 1], C), oracle.sign(y).reshape(y.shape))
        assert_close(K[n:n + 1], oracle.box_filter(oracle.channel_abs_mean(y), 3, 3, 1, 1), "K")


def test_static_scratch_rejects_sizes_beyond_its_array():
    """Checked on the host before anything touches the GPU, so this needs none."""
    lib = X.load()
    p, null = ctypes.c_void_p(0x1000), ctypes.c_void_p(0)
    too_big = X.make_desc(257, 64, 64, 64, 8, 3, 3, 1, 1)      # 257 * 4096 pixels > 2**20
    assert too_big.N * too_big.H * too_big.W > B.BINACTIV_STATIC_MAX_PIXELS
    assert lib.xnor_binactiv_static(p, null, null, ctypes.byref(too_big), p, p, null) == \
        B.XNOR_ERR_UNSUPPORTED
    ok = X.make_desc(1, 8, 5, 5, 4, 3, 3, 1, 1)
    assert lib.xnor_binactiv_static(null, null, null, ctypes.byref(ok), p, p, null) == \
        B.XNOR_ERR_INVALID_ARG
    assert lib.xnor_binactiv_static(p, null, null, ctypes.byref(ok), p, null, null) == \
        B.XNOR_ERR_INVALID_ARG
