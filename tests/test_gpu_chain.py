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
