"""Oracle parity on the code paths the benchmark times.

xnor_conv2d_forward picks its store path by its arguments: with acc_out = NULL (how bench.py and
the chain runner call it) the epilogue takes one of two lean branches (no residual / residual),
with acc_out it takes the general one.  The other parity files pass acc_out to compare the
integer sums; here every call passes acc_out = NULL and `out` is compared with the oracle
element by element, at the benchmark's batch sizes, on the images the oracle recomputes
(first, middle, last: images are independent through the whole block).  The integer sums of
the same shapes are proven on the other branch.
"""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from paper_1603_05279_b200 import workloads as wl
from paper_1603_05279_b200.runner import ChainRunner
from util import GuardSet, assert_close, dev, host, unpack_activations

pytestmark = pytest.mark.gpu


def _prepare(s, seed):
    x = wl.make_input(s, seed)
    w = wl.make_weights(s, seed)
    d = X.desc_of(s)
    wp, alpha = X.alloc_weights(s.C_out, s.C_in, s.k, s.k)
    xp, A, K = X.alloc_binactiv(d)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
    return x, w, d, wp, alpha, xp, K


def _images(N):
    return sorted({0, N // 2, N - 1})


def _check_out(oracle, s, x, w, out, images, residual=None, what=""):
    for n in images:
        res = None if residual is None else host(residual[n:n + 1])
        r = oracle.xnor_block(x[n:n + 1], w, s.stride, s.pad, residual=res)
        assert_close(host(out[n:n + 1]), r.out, "%s %s image %d" % (s.name, what, n))


LAYERS = [("alexnet", i) for i in range(len(wl.ALEXNET))] + [("resnet18", i) for i in range(len(wl.RESNET18))]


@pytest.mark.parametrize("config,li", LAYERS)
def test_layers_at_full_batch_without_acc_out(oracle, config, li):
    """Every AlexNet and ResNet layer at batch 256 through the two lean store branches: no
    residual; a residual in its own buffer; a residual that is the output buffer itself."""
    s = wl.CONFIGS[config][li]
    x, w, d, wp, alpha, xp, K = _prepare(s, wl.layer_seed(config, li))
    gs = GuardSet()
    out = gs.like("out", X.alloc_out(d))
    X.xnor_conv2d_forward(xp, wp, alpha, K, None, d, out, None)
    X.xnor_check_device()
    gs.check()
    _check_out(oracle, s, x, w, out, _images(s.N), what="plain")
    assert bool(torch.isfinite(out).all())

    res = torch.from_numpy(wl.normal(tuple(out.shape), 4242 + li)).cuda()
    out2 = gs.like("out_res", out)
    X.xnor_conv2d_forward(xp, wp, alpha, K, res, d, out2, None)
    X.xnor_check_device()
    gs.check()
    _check_out(oracle, s, x, w, out2, _images(s.N), residual=res, what="residual")
    # the two branches differ by the addition alone
    assert torch.equal(out2, out + res)

    out3 = res.clone()
    X.xnor_conv2d_forward(xp, wp, alpha, K, out3, d, out3, None)
    X.xnor_check_device()
    assert torch.equal(out3, out2)


@pytest.mark.parametrize("idx", range(len(wl.SWEEP)))
def test_every_sweep_point(oracle, idx):
    """All 24 (C_in, k) points of the efficiency sweep, as the benchmark runs them (batch 64,
    acc_out = NULL): the whole batch where the oracle needs under a second (<= 1 GMAC), else the
    first and the last image.  The integer sums are compared too, from a second call."""
    s = wl.SWEEP[idx]
    x, w, d, wp, alpha, xp, K = _prepare(s, wl.layer_seed("sweep", idx))
    out = X.alloc_out(d)
    X.xnor_conv2d_forward(xp, wp, alpha, K, None, d, out, None)
    acc = X.alloc_out(d, torch.int32)
    out_b = X.alloc_out(d)
    X.xnor_conv2d_forward(xp, wp, alpha, K, None, d, out_b, acc)
    X.xnor_check_device()
    assert torch.equal(out, out_b)
    images = [slice(0, s.N)] if wl.macs(s) <= 1e9 else [slice(0, 1), slice(s.N - 1, s.N)]
    for sl in images:
        r = oracle.xnor_block(x[sl], w, s.stride, s.pad)
        assert np.array_equal(host(acc[sl]), r.acc), s.name
        assert_close(host(out[sl]), r.out, s.name)


def _fill(ch, seed0):
    ch.x0.copy_(torch.from_numpy(wl.normal(tuple(ch.x0.shape), seed0)))
    for i, L in enumerate(ch.layers):
        L["w"].copy_(torch.from_numpy(wl.make_weights(L["shape"], seed0 + i)))
    for i, P in ch.proj.items():
        P["w"].copy_(torch.from_numpy(wl.normal(tuple(P["w"].shape), seed0 + 700 + i, 0.05)))


def _residual_of(ch, i):
    if i % 2 == 0:
        return None
    b0 = i - 1
    return ch.proj[b0]["out"] if b0 in ch.proj else ch.layer_input(b0)


def test_chain_at_benchmark_batch_without_acc_out(oracle):
    """The 16-layer chain exactly as bench.py --workload chain runs it (batch 256, no integer
    output), teacher-forced: the oracle of a layer starts from the GPU's own fp32 input and
    residual of that layer, first and last image."""
    ch = ChainRunner(256)
    _fill(ch, wl.layer_seed("chain", 0))
    ch.binarize_weights()
    ch.calibrate()
    ch.forward()
    X.xnor_check_device()
    for i, L in enumerate(ch.layers):
        s = L["shape"]
        for n in (0, 255):
            xin = host(ch.layer_input(i)[n:n + 1])
            res = _residual_of(ch, i)
            res = None if res is None else host(res[n:n + 1])
            r = oracle.xnor_block(xin, host(L["w"]), s.stride, s.pad, host(L["scale"]), host(L["shift"]), res)
            assert_close(host(L["out"][n:n + 1]), r.out, "layer %d image %d" % (i, n))


def test_fused_chain_at_benchmark_batch(oracle):
    """forward_fused at batch 256.  The fused run does not write the fp32 output of a block's
    first convolution, so for every layer that tensor is materialised by one plain call from the
    fused run's own inputs of the layer (same values bit for bit: asserted where the fused run
    did write it).  What the fused epilogue emitted for the next layer (packed bits, A, K) must
    be the oracle's BinActiv of that tensor; the tensor itself is tied to the oracle by teacher
    forcing from the previous one.  First and last image."""
    ch = ChainRunner(256)
    _fill(ch, wl.layer_seed("chain", 0))
    ch.binarize_weights()
    ch.calibrate()
    ch.prepare_fused()
    for L in ch.layers[1:]:
        L["x_packed"].zero_(); L["A"].fill_(float("nan")); L["K"].fill_(float("nan"))
    for L in ch.layers:
        L["out"].fill_(float("nan"))
    ch.forward_fused()
    X.xnor_check_device()
    prev = None                        # fp32 input of the current layer, as the GPU had it
    for i, L in enumerate(ch.layers):
        s = L["shape"]
        residual = _residual_of(ch, i)
        out = torch.empty_like(L["out"])
        X.xnor_conv2d_forward(L["x_packed"], L["w_packed"], L["alpha"], L["K"], residual, L["desc"], out, None)
        if i % 2 == 1:
            assert torch.equal(out, L["out"]), i
        else:
            assert bool(torch.isnan(L["out"]).all()), "the fused run does not write this tensor"
        xin = ch.x0 if i == 0 else prev
        for n in (0, 255):
            res = None if residual is None else host(residual[n:n + 1])
            r = oracle.xnor_block(host(xin[n:n + 1]), host(L["w"]), s.stride, s.pad, host(L["scale"]),
                                  host(L["shift"]), res)
            assert np.array_equal(unpack_activations(host(L["x_packed"][n:n + 1]), s.C_in), r.H), (i, n)
            assert_close(host(L["A"][n:n + 1]), r.A, "A of layer %d image %d" % (i, n))
            assert_close(host(L["K"][n:n + 1]), r.K, "K of layer %d image %d" % (i, n))
            assert_close(host(out[n:n + 1]), r.out, "out of layer %d image %d" % (i, n))
        prev = out


def test_binactiv_with_many_channels_and_pixels(oracle):
    """1024 channels with a BatchNorm affine on 65536 pixels: the shape at which the staged words
    of eight pixel groups no longer fit shared memory and the launcher spreads the channel
    words of a pixel group over the warps instead."""
    N, C, H, W = 256, 1024, 16, 16
    g = np.random.Generator(np.random.Philox(99))
    x = g.standard_normal((N, C, H, W), dtype=np.float32)
    scale = (1.0 + 0.1 * g.standard_normal(C)).astype(np.float32)
    shift = (0.1 * g.standard_normal(C)).astype(np.float32)
    d = X.make_desc(N, C, H, W, 8, 3, 3, 1, 1)
    gs = GuardSet()
    xp, A, K = (gs.like(n, t) for n, t in zip(("x_packed", "A", "K"), X.alloc_binactiv(d)))
    assert X.xnor_binactiv_launches(d, True) == 2
    X.xnor_binactiv(dev(x), dev(scale), dev(shift), d, xp, A, K)
    gs.check()
    for n in (0, 100, 255):
        y = oracle.bn_affine(x[n:n + 1], scale, shift)
        assert np.array_equal(unpack_activations(host(xp[n:n + 1]), C), oracle.sign(y).reshape(y.shape))
        A_or = oracle.channel_abs_mean(y)
        assert_close(host(A[n:n + 1]), A_or, "A")
        assert_close(host(K[n:n + 1]), oracle.box_filter(A_or, 3, 3, 1, 1), "K")
    # beyond what the kernels cover: refused on the host, nothing launched
    big = X.make_desc(2, 4000, 8, 8, 8, 3, 3, 1, 1)
    with pytest.raises(X.XnorError) as e:
        X.xnor_binactiv(torch.empty((2, 4000, 8, 8), device="cuda"), torch.ones(4000, device="cuda"),
                        torch.zeros(4000, device="cuda"), big, *X.alloc_binactiv(big))
    assert e.value.status == B.XNOR_ERR_UNSUPPORTED


# N, C, H, W, k, stride, pad, BatchNorm affine, flags
IMAGE_PATH_SHAPES = [
    (256, 96, 27, 27, 5, 1, 2, True, 0),            # AlexNet conv2's input: 8-channel chunks
    (200, 384, 13, 13, 3, 1, 1, False, 0),          # conv4 / conv5: 32-channel chunks
    (150, 40, 13, 13, 3, 2, 1, True, B.XNOR_FLAG_K_VALID_TAPS),   # a word with 8 channels only
    (96, 512, 7, 7, 3, 1, 1, True, 0),              # ResNet's last stage
    (80, 8, 31, 33, 7, 2, 3, True, 0),              # 1023 pixels: one chunk per image
    (300, 24, 5, 9, 1, 1, 0, False, 0),             # more images than resident blocks
]


@pytest.mark.parametrize("shape", IMAGE_PATH_SHAPES)
def test_binactiv_on_planes_of_odd_size_with_many_images(oracle, shape):
    """Inputs whose planes are not a multiple of four pixels, with enough images to occupy the
    GPU, go through the kernel that streams whole images with bulk copies and forms K in the same
    launch: bits identical, A and K within tolerance, on the first, middle and last images and
    on the one after the first round of blocks; nothing written outside the outputs."""
    N, C, H, W, k, stride, pad, bn, flags = shape
    g = np.random.Generator(np.random.Philox(sum(shape[:7])))
    x = g.standard_normal((N, C, H, W), dtype=np.float32)
    scale = (1.0 + 0.2 * g.standard_normal(C)).astype(np.float32) if bn else None
    shift = (0.2 * g.standard_normal(C)).astype(np.float32) if bn else None
    d = X.make_desc(N, C, H, W, 8, k, k, stride, pad, flags)
    gs = GuardSet()
    xp, A, K = (gs.like(n, t) for n, t in zip(("x_packed", "A", "K"), X.alloc_binactiv(d)))
    xp.fill_(-1); A.fill_(float("nan")); K.fill_(float("nan"))
    xd = dev(x)
    sc, sh = (None, None) if scale is None else (dev(scale), dev(shift))
    assert X.xnor_binactiv_launches(d, bn) == 1
    X.xnor_binactiv(xd, sc, sh, d, xp, A, K)
    X.xnor_check_device()
    gs.check()
    assert bool(torch.isfinite(A).all()) and bool(torch.isfinite(K).all())
    # a few images alone take the two-kernel path: same bits
    d8 = X.make_desc(8, C, H, W, 8, k, k, stride, pad, flags)
    assert X.xnor_binactiv_launches(d8, bn) == 2
    xp2, A2, K2 = X.alloc_binactiv(d8)
    X.xnor_binactiv(xd[N - 8:].contiguous(), sc, sh, d8, xp2, A2, K2)
    assert torch.equal(xp2, xp[N - 8:])
    assert_close(host(A2), host(A[N - 8:]), "A of the two paths")
    assert_close(host(K2), host(K[N - 8:]), "K of the two paths")
    for n in sorted({0, 1, N // 2, min(N - 1, 296), N - 1}):
        y = x[n:n + 1] if scale is None else oracle.bn_affine(x[n:n + 1], scale, shift)
        assert np.array_equal(unpack_activations(host(xp[n:n + 1]), C), oracle.sign(y).reshape(y.shape)), n
        A_or = oracle.channel_abs_mean(y)
        assert_close(host(A[n:n + 1]), A_or, "A of image %d" % n)
        K_or = (oracle.box_filter_valid_taps if flags & B.XNOR_FLAG_K_VALID_TAPS else oracle.box_filter)(
            A_or, k, k, stride, pad)
        assert_close(host(K[n:n + 1]), K_or, "K of image %d" % n)
    # bits of channels beyond C_in in the last word are zero, as from the other BinActiv kernel
    if C % 32:
        assert int((xp[..., -1].to(torch.int64) & 0xFFFFFFFF).max()) < (1 << (C % 32))
