"""GPU parity: libxnor (through its C ABI) against the CPU oracle, element by
element, on the same seeded inputs.  Integer and bit results must be identical;
fp32 results within REL_TOL of the tensor's largest magnitude."""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from paper_1603_05279_b200 import workloads as wl
from util import REL_TOL, GuardSet, assert_close, dev, host, unpack_activations, unpack_weights

pytestmark = pytest.mark.gpu

ENGINES = [B.XNOR_ENGINE_POPC, B.XNOR_ENGINE_UMMA, B.XNOR_ENGINE_UMMA_STREAM, B.XNOR_ENGINE_UMMA_SINGLE,
           B.XNOR_ENGINE_UMMA_PAIR, B.XNOR_ENGINE_UMMA_PAIR_STREAM, B.XNOR_ENGINE_AUTO]
TC_ENGINES = (B.XNOR_ENGINE_UMMA, B.XNOR_ENGINE_UMMA_STREAM, B.XNOR_ENGINE_UMMA_SINGLE,
              B.XNOR_ENGINE_UMMA_PAIR, B.XNOR_ENGINE_UMMA_PAIR_STREAM)


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def gpu_block(x, w, stride, pad, scale=None, shift=None, residual=None, engine=B.XNOR_ENGINE_AUTO,
              alias_residual=False):
    """Runs binarize_weights -> binactiv -> conv2d_forward on the GPU; returns host arrays."""
    N, C, H, W = x.shape
    Co, _, kh, kw = w.shape
    d = X.make_desc(N, C, H, W, Co, kh, kw, stride, pad)
    # every output lies between guard words that must survive the calls
    gs = GuardSet()
    wp0, alpha0 = X.alloc_weights(Co, C, kh, kw)
    xp0, A0, K0 = X.alloc_binactiv(d)
    wp, alpha = gs.like("w_packed", wp0), gs.like("alpha", alpha0)
    xp, A, K = gs.like("x_packed", xp0), gs.like("A", A0), gs.like("K", K0)
    out = gs.like("out", X.alloc_out(d))
    acc = gs.like("acc_out", X.alloc_out(d, torch.int32))
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None if scale is None else dev(scale),
                    None if shift is None else dev(shift), d, xp, A, K)
    res = None
    if residual is not None:
        if alias_residual:
            out.copy_(dev(residual))
            res = out
        else:
            res = dev(residual)
    X.xnor_set_engine(engine)
    try:
        X.xnor_conv2d_forward(xp, wp, alpha, K, res, d, out, acc)
    finally:
        X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
    X.xnor_check_device()
    gs.check()
    return dict(wp=host(wp), alpha=host(alpha), xp=host(xp), A=host(A), K=host(K),
                out=host(out), acc=host(acc))


def check_block(oracle, x, w, stride, pad, scale=None, shift=None, residual=None,
                engine=B.XNOR_ENGINE_AUTO, alias_residual=False):
    g = gpu_block(x, w, stride, pad, scale, shift, residual, engine, alias_residual)
    r = oracle.xnor_block(x, w, stride, pad, scale, shift, residual)
    C = x.shape[1]
    assert np.array_equal(unpack_weights(g["wp"], C, w.shape[2], w.shape[3]), r.B), "sign(W) bits"
    assert np.array_equal(unpack_activations(g["xp"], C), r.H), "sign(I) bits"
    assert_close(g["alpha"], r.alpha, "alpha")
    assert_close(g["A"], r.A, "A")
    assert_close(g["K"], r.K, "K")
    assert np.array_equal(g["acc"], r.acc), "integer accumulators must be bit-exact"
    assert_close(g["out"], r.out, "out")
    return g, r


SHAPES = [
    # N, C, H, W, Co, kh, kw, stride, pad
    (1, 64, 14, 14, 64, 3, 3, 1, 1),      # the single-layer configuration
    (2, 3, 9, 11, 5, 3, 3, 1, 1),         # fewer than 32 channels, odd sizes
    (3, 96, 13, 13, 70, 5, 5, 1, 2),      # 3 words, C_out not a multiple of the filter tile
    (2, 100, 7, 7, 33, 3, 3, 1, 1),       # channel tail inside the last word
    (2, 64, 17, 15, 64, 3, 3, 2, 1),      # stride 2, ragged
    (2, 32, 14, 14, 64, 1, 1, 1, 0),      # 1x1
    (1, 40, 14, 14, 16, 7, 7, 1, 3),      # 7x7
    (2, 64, 8, 8, 32, 3, 3, 1, 0),        # no padding
    (1, 64, 6, 9, 8, 3, 2, 1, 1),         # rectangular filter
    (2, 33, 10, 10, 9, 3, 3, 2, 0),       # stride 2 without padding
    (1, 8, 1, 1, 4, 1, 1, 1, 0),          # one pixel
    (2, 16, 5, 5, 4, 5, 5, 1, 3),         # pad larger than k/2
    (1, 288, 9, 9, 130, 3, 3, 1, 1),      # 9 words (more than one shared-memory chunk)
    (2, 16, 12, 12, 12, 3, 3, 3, 1),      # stride 3
]


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("shape", SHAPES)
def test_block_parity(oracle, shape, engine):
    N, C, H, W, Co, kh, kw, s, p = shape
    g = rng(sum(shape))
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, kh, kw)).astype(np.float32)
    if engine in TC_ENGINES and s > 2:
        with pytest.raises(X.XnorError) as e:       # strides a tensor-core engine does not cover
            gpu_block(x, w, s, p, engine=engine)
        assert e.value.status == B.XNOR_ERR_UNSUPPORTED
        return
    check_block(oracle, x, w, s, p, engine=engine)


@pytest.mark.parametrize("engine", ENGINES)
def test_block_parity_with_bn_and_residual(oracle, engine):
    g = rng(5)
    N, C, H, W, Co = 3, 70, 13, 13, 40
    x = (2.0 + 3.0 * g.standard_normal((N, C, H, W))).astype(np.float32)
    w = (0.05 * g.standard_normal((Co, C, 3, 3))).astype(np.float32)
    scale = (1.0 / 3.0 + 0.05 * g.standard_normal(C)).astype(np.float32)
    shift = (-2.0 / 3.0 + 0.05 * g.standard_normal(C)).astype(np.float32)
    res = g.standard_normal((N, Co, H, W)).astype(np.float32)
    check_block(oracle, x, w, 1, 1, scale, shift, res, engine=engine)
    check_block(oracle, x, w, 1, 1, scale, shift, res, engine=engine, alias_residual=True)


def test_zeros_and_negative_zero_are_plus_one(oracle):
    g = rng(6)
    x = g.standard_normal((2, 40, 6, 6)).astype(np.float32)
    x[0, :, 2, 3] = 0.0
    x[1, ::2, 1, 1] = -0.0
    w = g.standard_normal((8, 40, 3, 3)).astype(np.float32)
    w[3, :, 1, 1] = 0.0
    w[4, ::3] = -0.0
    gpu, _ = check_block(oracle, x, w, 1, 1)
    assert (unpack_activations(gpu["xp"], 40)[0, :, 2, 3] == 1).all()


def test_bn_sign_decisions_use_one_fused_rounding(oracle):
    """Inputs placed so that scale*x + shift is within an ulp of zero: the sign
    bits still agree with the oracle because both sides use one fmaf."""
    g = rng(7)
    C = 48
    scale = (1.0 + 0.5 * g.random(C)).astype(np.float32)
    x = g.standard_normal((2, C, 8, 8)).astype(np.float32)
    shift = (-scale * x[0, :, 0, 0]).astype(np.float32)     # y ~ 0 at (0,:,0,0)
    x[1] = x[0] * (1 + 1e-7)
    w = g.standard_normal((8, C, 3, 3)).astype(np.float32)
    check_block(oracle, x, w, 1, 1, scale, shift)


def test_constant_magnitude_inputs_give_the_dense_convolution(oracle):
    """Eq. 10 with equality: x in {+-c1}, w in {+-c2} -> the GPU block equals the
    dense convolution where the window is inside the image."""
    import torch.nn.functional as F
    g = rng(8)
    x = np.where(g.random((2, 64, 10, 10)) < 0.5, -0.5, 0.5).astype(np.float32)
    w = np.where(g.random((16, 64, 3, 3)) < 0.5, -0.25, 0.25).astype(np.float32)
    gpu = gpu_block(x, w, 1, 0)
    dense = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double()).numpy()
    assert np.array_equal(gpu["out"].astype(np.float64), dense)


def test_shortcut_conv_parity(oracle):
    g = rng(9)
    # the ResNet shape; odd sizes (channel and filter tails, pixel tiles that straddle images,
    # H_out*W_out not a multiple of 4); a 7x7 output at batch 40 (several tiles over many images)
    for (N, C, H, W, Co, s) in [(2, 64, 56, 56, 128, 2), (3, 70, 9, 7, 33, 2), (1, 16, 5, 5, 8, 1),
                                (40, 256, 14, 14, 130, 2), (5, 36, 6, 6, 64, 1), (7, 3, 1, 1, 2, 1)]:
        x = g.standard_normal((N, C, H, W)).astype(np.float32)
        w = (0.05 * g.standard_normal((Co, C))).astype(np.float32)
        out = torch.empty((N, Co, (H - 1) // s + 1, (W - 1) // s + 1), device="cuda")
        X.xnor_shortcut_conv1x1(dev(x), dev(w), s, out)
        assert_close(host(out), oracle.shortcut_conv1x1(x, w.reshape(Co, C, 1, 1), s), "shortcut")


# ------------------------------------------------------------------ named workloads
def _run_layer_full(s, seed, engine=B.XNOR_ENGINE_AUTO):
    x = wl.make_input(s, seed)
    w = wl.make_weights(s, seed)
    d = X.desc_of(s)
    wp, alpha = X.alloc_weights(s.C_out, s.C_in, s.k, s.k)
    xp, A, K = X.alloc_binactiv(d)
    out = X.alloc_out(d)
    acc = X.alloc_out(d, torch.int32)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
    X.xnor_set_engine(engine)
    try:
        X.xnor_conv2d_forward(xp, wp, alpha, K, None, d, out, acc)
    finally:
        X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
    X.xnor_check_device()
    torch.cuda.synchronize()
    return x, w, out, acc, K


def _check_sampled_images(oracle, s, x, w, out, acc, images):
    """Images are independent through the whole block: the oracle recomputes the
    chosen images from the same inputs."""
    for n in images:
        r = oracle.xnor_block(x[n:n + 1], w, s.stride, s.pad)
        assert np.array_equal(host(acc[n:n + 1]), r.acc), (s.name, n)
        assert_close(host(out[n:n + 1]), r.out, "%s image %d" % (s.name, n))


def test_single_layer_configuration(oracle):
    s = wl.SINGLE[0]
    x, w, out, acc, _ = _run_layer_full(s, wl.layer_seed("single", 0))
    _check_sampled_images(oracle, s, x, w, out, acc, [0])


@pytest.mark.parametrize("li", range(len(wl.ALEXNET)))
def test_alexnet_layers_at_full_batch(oracle, li):
    """The benchmark's own launch configuration (batch 256); first and last image
    recomputed by the oracle, plus invariants on every output."""
    s = wl.ALEXNET[li]
    x, w, out, acc, K = _run_layer_full(s, wl.layer_seed("alexnet", li))
    _check_sampled_images(oracle, s, x, w, out, acc, [0, s.N - 1])
    nmax = s.C_in * s.k * s.k
    a = acc.view(-1)
    assert int(a.abs().max()) <= nmax
    inner = acc[:, :, s.pad:-s.pad, s.pad:-s.pad]
    assert bool(((inner - nmax) % 2 == 0).all())          # parity of a full window
    assert bool(torch.isfinite(out).all())


@pytest.mark.parametrize("li,engine", [(0, B.XNOR_ENGINE_UMMA_STREAM), (0, B.XNOR_ENGINE_UMMA_PAIR),
                                       (1, B.XNOR_ENGINE_UMMA_PAIR_STREAM), (2, B.XNOR_ENGINE_UMMA_SINGLE),
                                       (2, B.XNOR_ENGINE_UMMA_PAIR), (3, B.XNOR_ENGINE_UMMA_PAIR_STREAM)])
def test_alexnet_layers_at_full_batch_pinned_variants(oracle, li, engine):
    """Every schedule of the tensor-core engine at the benchmark's size: CTAs whose item range
    crosses a slab boundary (a second fill of the resident slab), many rounds of every barrier,
    pairs with an odd number of stream tiles."""
    s = wl.ALEXNET[li]
    x, w, out, acc, K = _run_layer_full(s, wl.layer_seed("alexnet", li), engine)
    _check_sampled_images(oracle, s, x, w, out, acc, [0, s.N // 2, s.N - 1])


def test_engines_agree_bit_for_bit_on_odd_sizes():
    """All engines compute the same integers and apply the same two fp32 roundings, so their
    outputs are identical; shapes chosen for ragged tiles (odd pixel and filter counts, a
    channel tail, stride 2, one stream tile for a pair)."""
    for (N, C, H, W, Co, k, st, pad) in [(3, 70, 9, 7, 50, 3, 1, 1), (2, 40, 11, 11, 130, 5, 2, 2),
                                         (1, 33, 6, 5, 17, 3, 1, 0), (5, 200, 14, 14, 272, 3, 1, 1)]:
        g = rng(N * 1000 + C)
        s = wl.ConvShape("t", N, C, H, W, Co, k, st, pad, 1.0)
        x = g.standard_normal((N, C, H, W)).astype(np.float32)
        w = g.standard_normal((Co, C, k, k)).astype(np.float32)
        d = X.desc_of(s)
        wp, alpha = X.alloc_weights(Co, C, k, k)
        xp, A, K = X.alloc_binactiv(d)
        X.xnor_binarize_weights(dev(w), wp, alpha)
        X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
        outs = []
        for engine in ENGINES:
            out = X.alloc_out(d)
            X.xnor_set_engine(engine)
            try:
                X.xnor_conv2d_forward(xp, wp, alpha, K, None, d, out, None)
            finally:
                X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
            X.xnor_check_device()
            outs.append(out)
        for out in outs[1:]:
            assert torch.equal(out, outs[0])


def _random_shapes(count, seed):
    """Seeded shapes that walk the planner's corners: few or many channel words (the patch
    builders' cooperative mode starts at 12), filter counts around the slab widths, one or many
    pixel tiles, both strides, with and without padding."""
    g = rng(seed)
    shapes = []
    while len(shapes) < count:
        C = int(g.choice([1, 31, 64, 96, 200, 384, 400, 520]))
        Co = int(g.choice([1, 16, 40, 129, 224, 256, 300]))
        k = int(g.choice([1, 2, 3, 5]))
        st = int(g.choice([1, 2]))
        pad = int(g.integers(0, k))
        H = int(g.integers(max(1, k - 2 * pad), 23))
        W = int(g.integers(max(1, k - 2 * pad), 23))
        N = int(g.choice([1, 2, 5, 19]))
        if C * k * k > 6000 and N * H * W > 2000:
            N = 1                                     # keep the popcount reference quick
        shapes.append((N, C, H, W, Co, k, st, pad))
    return shapes


@pytest.mark.parametrize("shape", _random_shapes(24, 20240607))
def test_tensor_core_variants_match_the_popcount_engine(shape):
    """The CUDA-core engine shares no code with the tensor-core kernels beyond the packed
    operands; integers and the two fp32 roundings are the same, so outputs must be identical."""
    N, C, H, W, Co, k, st, pad = shape
    g = rng(sum(shape))
    x = g.standard_normal((N, C, H, W)).astype(np.float32)
    w = g.standard_normal((Co, C, k, k)).astype(np.float32)
    res = g.standard_normal((N, Co, (H + 2 * pad - k) // st + 1, (W + 2 * pad - k) // st + 1)).astype(np.float32)
    d = B.xnor_conv_desc(N, C, H, W, Co, k, k, st, pad)
    wp, alpha = X.alloc_weights(Co, C, k, k)
    xp, A, K = X.alloc_binactiv(d)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
    r = dev(res)
    ref = None
    for engine in ENGINES:
        out = X.alloc_out(d)
        acc = X.alloc_out(d, torch.int32)
        X.xnor_set_engine(engine)
        try:
            X.xnor_conv2d_forward(xp, wp, alpha, K, r, d, out, acc)
        except X.XnorError as e:
            assert engine in TC_ENGINES and e.status == B.XNOR_ERR_UNSUPPORTED, (shape, engine)
            continue
        finally:
            X.xnor_set_engine(B.XNOR_ENGINE_AUTO)
        X.xnor_check_device()
        if ref is None:
            ref = (out, acc)
        else:
            assert torch.equal(acc, ref[1]), (shape, engine)
            assert torch.equal(out, ref[0]), (shape, engine)


@pytest.mark.parametrize("li", range(len(wl.RESNET18)))
def test_resnet_layers_at_full_batch(oracle, li):
    s = wl.RESNET18[li]
    x, w, out, acc, K = _run_layer_full(s, wl.layer_seed("resnet18", li))
    _check_sampled_images(oracle, s, x, w, out, acc, [s.N - 1])
    assert int(acc.abs().max()) <= s.C_in * s.k * s.k


@pytest.mark.parametrize("ci,k", [(32, 1), (64, 7), (1024, 3), (512, 5)])
def test_sweep_points(oracle, ci, k):
    s = [t for t in wl.SWEEP if t.C_in == ci and t.k == k][0]
    x, w, out, acc, K = _run_layer_full(s, wl.layer_seed("sweep", wl.SWEEP.index(s)))
    _check_sampled_images(oracle, s, x, w, out, acc, [0, s.N - 1])


def test_rel_tol_is_the_stated_one():
    assert REL_TOL == 1e-5
