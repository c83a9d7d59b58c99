"""The 16-layer ResNet-18 chain on the GPU against the oracle, layer by layer.

Teacher forcing: the oracle of layer i is fed the GPU's own fp32 input of that
layer (and the GPU's residual), so both sides binarise identical bits and the
integer sums must be identical; fp32 outputs within REL_TOL.  A free-running
end-to-end comparison would differ wherever a pre-sign value lies within
rounding of zero, which says nothing about either side."""
import numpy as np
import pytest
import torch

from paper_1603_05279_b200 import workloads as wl
from paper_1603_05279_b200.runner import ChainRunner
import paper_1603_05279_b200 as X
from util import assert_close, host

pytestmark = pytest.mark.gpu


def _fill(ch, seed0):
    ch.x0.copy_(torch.from_numpy(wl.normal(tuple(ch.x0.shape), seed0)))
    for i, L in enumerate(ch.layers):
        L["w"].copy_(torch.from_numpy(wl.make_weights(L["shape"], seed0 + i)))
    for i, P in ch.proj.items():
        P["w"].copy_(torch.from_numpy(wl.normal(tuple(P["w"].shape), seed0 + 700 + i, 0.05)))


def _check_layers(oracle, ch, images):
    for i, L in enumerate(ch.layers):
        s = L["shape"]
        x = host(ch.layer_input(i))[images]
        res = None
        if i % 2 == 1:
            b0 = i - 1
            if b0 in ch.proj:
                xin = host(ch.layer_input(b0))[images]
                pw = host(ch.proj[b0]["w"])
                res_or = oracle.shortcut_conv1x1(xin, pw.reshape(pw.shape[0], pw.shape[1], 1, 1),
                                                 ch.shapes[b0].stride)
                res = host(ch.proj[b0]["out"])[images]
                assert_close(res, res_or, "layer %d projection shortcut" % i)
            else:
                res = host(ch.layer_input(b0))[images]
        r = oracle.xnor_block(x, host(L["w"]), s.stride, s.pad, host(L["scale"]),
                              host(L["shift"]), res)
        assert np.array_equal(host(L["acc"])[images], r.acc), "layer %d integer sums" % i
        assert_close(host(L["out"])[images], r.out, "layer %d out" % i)


def test_chain_small_batch_every_image(oracle):
    ch = ChainRunner(2, keep_acc=True)
    _fill(ch, wl.layer_seed("chain", 0))
    ch.binarize_weights()
    ch.calibrate()
    ch.forward()
    X.xnor_check_device()
    # calibrated BatchNorm: the post-BN tensor of a middle layer is zero-mean, unit-variance
    L = ch.layers[5]
    y = ch.layer_input(5).double() * L["scale"].double()[None, :, None, None] + \
        L["shift"].double()[None, :, None, None]
    assert float(y.mean(dim=(0, 2, 3)).abs().max()) < 1e-4
    assert float((y.var(dim=(0, 2, 3), unbiased=False) - 1).abs().max()) < 1e-3
    assert bool(torch.isfinite(ch.layers[-1]["out"]).all())
    _check_layers(oracle, ch, [0, 1])


def test_chain_benchmark_batch_sampled_images(oracle):
    """The launch configuration bench.py --workload chain times (batch 256); the oracle
    recomputes the last image of every layer."""
    ch = ChainRunner(256, keep_acc=True)
    _fill(ch, wl.layer_seed("chain", 0))
    ch.binarize_weights()
    ch.calibrate()
    ch.forward()
    X.xnor_check_device()
    _check_layers(oracle, ch, [255])
    for L in ch.layers:
        s = L["shape"]
        assert int(L["acc"].abs().max()) <= s.C_in * 9


def test_fused_chain_is_consistent_with_the_plain_calls_layer_by_layer():
    """The chain with BinActiv fused into every BinConv.  Parity of the fused call with the
    oracle is established per layer elsewhere; here every fused layer of the running chain is
    re-done with the two plain calls from the same inputs: the fp32 output (where the chain
    keeps it) and the packed bits must be identical, A and K within the tolerance."""
    N = 4
    ch = ChainRunner(N)
    g = np.random.Generator(np.random.Philox(2024))
    ch.x0.copy_(torch.from_numpy(g.standard_normal(tuple(ch.x0.shape)).astype(np.float32)))
    for L in ch.layers:
        L["w"].copy_(torch.from_numpy((0.05 * g.standard_normal(tuple(L["w"].shape))).astype(np.float32)))
    for P in ch.proj.values():
        P["w"].copy_(torch.from_numpy((0.05 * g.standard_normal(tuple(P["w"].shape))).astype(np.float32)))
    ch.binarize_weights()
    ch.calibrate()
    ch.prepare_fused()
    assert sum(1 for p in ch.fused_parts if p > 0) == len(ch.layers) - 1
    ch.forward_fused()
    X.xnor_check_device()
    for i, L in enumerate(ch.layers[:-1]):
        nxt = ch.layers[i + 1]
        residual = None
        if i % 2 == 1:
            b0 = i - 1
            residual = ch.proj[b0]["out"] if b0 in ch.proj else ch.layer_input(b0)
        out = torch.empty_like(L["out"])
        X.xnor_conv2d_forward(L["x_packed"], L["w_packed"], L["alpha"], L["K"], residual, L["desc"], out, None)
        if i % 2 == 1:
            assert torch.equal(out, L["out"]), i
        xp, A, K = X.alloc_binactiv(nxt["desc"])
        X.xnor_binactiv(out, nxt["scale"], nxt["shift"], nxt["desc"], xp, A, K)
        assert torch.equal(xp, nxt["x_packed"]), i
        assert_close(host(nxt["A"]), host(A), "A of layer %d" % (i + 1))
        assert_close(host(nxt["K"]), host(K), "K of layer %d" % (i + 1))
