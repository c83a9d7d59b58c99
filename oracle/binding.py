"""ctypes binding of the C oracle (test infrastructure; holds no arithmetic).

Every function takes and returns C-contiguous numpy arrays and forwards to the
C routine of the same name in ``xnor_oracle.c``.
"""
import ctypes
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xnor_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def lib_path():
    return _LIB


def build(force=False):
    """Compile xnor_oracle.c into liboracle.so beside it (gcc, OpenMP)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fno-fast-math", "-ffp-contract=off",
           "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_speedup_model.restype = ctypes.c_double
        _lib.oracle_speedup_model.argtypes = [ctypes.c_double, ctypes.c_double]
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _i(*v):
    return [ctypes.c_int(int(t)) for t in v]


def out_extent(n, k, stride, pad):
    return (n + 2 * pad - k) // stride + 1


def num_threads():
    return int(_load().oracle_num_threads())


def set_num_threads(n):
    _load().oracle_set_num_threads(ctypes.c_int(int(n)))


def bn_affine(x, scale, shift):
    x = _f32(x)
    N, C, H, W = x.shape
    scale, shift = _f32(scale), _f32(shift)
    y = np.empty_like(x)
    _load().oracle_bn_affine(_p(x), _p(scale), _p(shift), *_i(N, C, H, W), _p(y))
    return y


def sign(v):
    v = _f32(v)
    s = np.empty(v.shape, dtype=np.int8)
    _load().oracle_sign(_p(v), ctypes.c_size_t(v.size), _p(s))
    return s


def channel_abs_mean(y):
    y = _f32(y)
    N, C, H, W = y.shape
    A = np.empty((N, H, W), dtype=np.float32)
    _load().oracle_channel_abs_mean(_p(y), *_i(N, C, H, W), _p(A))
    return A


def box_filter(A, kh, kw, stride, pad):
    A = _f32(A)
    N, H, W = A.shape
    K = np.empty((N, out_extent(H, kh, stride, pad), out_extent(W, kw, stride, pad)),
                 dtype=np.float32)
    _load().oracle_box_filter(_p(A), *_i(N, H, W, kh, kw, stride, pad), _p(K))
    return K


def binarize_weights(w):
    w = _f32(w)
    Co, C, kh, kw = w.shape
    B = np.empty(w.shape, dtype=np.int8)
    alpha = np.empty((Co,), dtype=np.float32)
    _load().oracle_binarize_weights(_p(w), *_i(Co, C, kh, kw), _p(B), _p(alpha))
    return B, alpha


def binconv_acc(Hs, B, stride, pad):
    Hs = np.ascontiguousarray(Hs, dtype=np.int8)
    B = np.ascontiguousarray(B, dtype=np.int8)
    N, C, H, W = Hs.shape
    Co, C2, kh, kw = B.shape
    assert C == C2
    acc = np.empty((N, Co, out_extent(H, kh, stride, pad), out_extent(W, kw, stride, pad)),
                   dtype=np.int32)
    _load().oracle_binconv_acc(_p(Hs), _p(B), *_i(N, C, H, W, Co, kh, kw, stride, pad), _p(acc))
    return acc


def scale_output(acc, K, alpha, residual=None):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    K, alpha, residual = _f32(K), _f32(alpha), _f32(residual)
    N, Co, Ho, Wo = acc.shape
    out = np.empty(acc.shape, dtype=np.float32)
    _load().oracle_scale_output(_p(acc), _p(K), _p(alpha), _p(residual), *_i(N, Co, Ho, Wo), _p(out))
    return out


def xnor_block(x, w, stride, pad, bn_scale=None, bn_shift=None, residual=None):
    """BN -> BinActiv -> BinConv; returns every intermediate by name."""
    x, w = _f32(x), _f32(w)
    bn_scale, bn_shift, residual = _f32(bn_scale), _f32(bn_shift), _f32(residual)
    N, C, H, W = x.shape
    Co, C2, kh, kw = w.shape
    assert C == C2
    Ho, Wo = out_extent(H, kh, stride, pad), out_extent(W, kw, stride, pad)
    r = SimpleNamespace(
        y=np.empty_like(x), H=np.empty(x.shape, np.int8), A=np.empty((N, H, W), np.float32),
        K=np.empty((N, Ho, Wo), np.float32), B=np.empty(w.shape, np.int8),
        alpha=np.empty((Co,), np.float32), acc=np.empty((N, Co, Ho, Wo), np.int32),
        out=np.empty((N, Co, Ho, Wo), np.float32))
    _load().oracle_xnor_block(_p(x), _p(bn_scale), _p(bn_shift), _p(w), _p(residual),
                              *_i(N, C, H, W, Co, kh, kw, stride, pad),
                              _p(r.y), _p(r.H), _p(r.A), _p(r.K), _p(r.B), _p(r.alpha),
                              _p(r.acc), _p(r.out))
    return r


def xnor_block_ex(x, w, stride, pad, bn_scale=None, bn_shift=None, residual=None, kbits=1,
                  relu=False, k_valid_taps=False):
    """The block with its options (k-bit activations, ReLU, border variant of K)."""
    x, w = _f32(x), _f32(w)
    bn_scale, bn_shift, residual = _f32(bn_scale), _f32(bn_shift), _f32(residual)
    N, C, H, W = x.shape
    Co, C2, kh, kw = w.shape
    assert C == C2
    Ho, Wo = out_extent(H, kh, stride, pad), out_extent(W, kw, stride, pad)
    r = SimpleNamespace(
        y=np.empty_like(x), H=np.empty(x.shape, np.int8), A=np.empty((N, H, W), np.float32),
        K=np.empty((N, Ho, Wo), np.float32), B=np.empty(w.shape, np.int8),
        alpha=np.empty((Co,), np.float32), acc=np.empty((N, Co, Ho, Wo), np.int32),
        out=np.empty((N, Co, Ho, Wo), np.float32))
    _load().oracle_xnor_block_ex(_p(x), _p(bn_scale), _p(bn_shift), _p(w), _p(residual),
                                 *_i(N, C, H, W, Co, kh, kw, stride, pad, kbits,
                                     1 if relu else 0, 1 if k_valid_taps else 0),
                                 _p(r.y), _p(r.H), _p(r.A), _p(r.K), _p(r.B), _p(r.alpha),
                                 _p(r.acc), _p(r.out))
    return r


def box_filter_valid_taps(A, kh, kw, stride, pad):
    A = _f32(A)
    N, H, W = A.shape
    K = np.empty((N, out_extent(H, kh, stride, pad), out_extent(W, kw, stride, pad)),
                 dtype=np.float32)
    _load().oracle_box_filter_valid_taps(_p(A), *_i(N, H, W, kh, kw, stride, pad), _p(K))
    return K


def relu(v):
    r = np.array(_f32(v), copy=True, order="C")
    _load().oracle_relu(_p(r), ctypes.c_size_t(r.size))
    return r


def quantize_k(v, k):
    """Level codes L of q_k (odd integers in [-(2^k-1), 2^k-1]); the level is L / (2^k - 1)."""
    v = _f32(v)
    L = np.empty(v.shape, dtype=np.int8)
    _load().oracle_quantize_k(_p(v), ctypes.c_size_t(v.size), ctypes.c_int(int(k)), _p(L))
    return L


def scale_output_k(acc, k, K, alpha, residual=None):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    K, alpha, residual = _f32(K), _f32(alpha), _f32(residual)
    N, Co, Ho, Wo = acc.shape
    out = np.empty(acc.shape, dtype=np.float32)
    _load().oracle_scale_output_k(_p(acc), ctypes.c_int(int(k)), _p(K), _p(alpha), _p(residual),
                                  *_i(N, Co, Ho, Wo), _p(out))
    return out


def round_bf16(v):
    v = _f32(v)
    r = np.empty_like(v)
    _load().oracle_round_bf16(_p(v), ctypes.c_size_t(v.size), _p(r))
    return r


def bwn_conv(x, B, alpha, stride, pad, residual=None):
    """Binary-Weight-Network convolution (I (+) B) alpha on real inputs x (Eq. 1)."""
    x, alpha, residual = _f32(x), _f32(alpha), _f32(residual)
    B = np.ascontiguousarray(B, dtype=np.int8)
    N, C, H, W = x.shape
    Co, C2, kh, kw = B.shape
    assert C == C2
    out = np.empty((N, Co, out_extent(H, kh, stride, pad), out_extent(W, kw, stride, pad)), np.float32)
    _load().oracle_bwn_conv(_p(x), _p(B), _p(alpha), _p(residual),
                            *_i(N, C, H, W, Co, kh, kw, stride, pad), _p(out))
    return out


def binary_gradient_backward(g, B, alpha, pad, in_hw, round_products=False):
    """Backward convolution with the gradient binarised to gmax * sign(g) and the filters
    alpha * B (Section 3.2, "Binary Gradient"), stride 1.  g [N][Co][Ho][Wo], B [Co][C][kh][kw];
    returns (gmax [N], gin [N][C][H][W])."""
    g, alpha = _f32(g), _f32(alpha)
    B = np.ascontiguousarray(B, dtype=np.int8)
    N, Co, Ho, Wo = g.shape
    Co2, C, kh, kw = B.shape
    H, W = in_hw
    assert Co == Co2 and Ho == out_extent(H, kh, 1, pad) and Wo == out_extent(W, kw, 1, pad)
    gmax = np.empty((N,), np.float32)
    gin = np.empty((N, C, H, W), np.float32)
    _load().oracle_binary_gradient_backward(_p(g), _p(B), _p(alpha), *_i(N, C, H, W, Co, kh, kw, pad),
                                            ctypes.c_int(1 if round_products else 0), _p(gmax), _p(gin))
    return gmax, gin


def shortcut_conv1x1(x, w, stride):
    x, w = _f32(x), _f32(w)
    N, C, H, W = x.shape
    Co = w.shape[0]
    w2 = np.ascontiguousarray(w.reshape(Co, C))
    out = np.empty((N, Co, (H - 1) // stride + 1, (W - 1) // stride + 1), np.float32)
    _load().oracle_shortcut_conv1x1(_p(x), _p(w2), *_i(N, C, H, W, Co, stride), _p(out))
    return out


def maxpool2d(x, k, stride, pad=0, relu=False):
    """Max pooling (optionally after ReLU) of an NCHW fp32 tensor; padding taps take no part."""
    x = _f32(x)
    N, C, H, W = x.shape
    out = np.empty((N, C, out_extent(H, k, stride, pad), out_extent(W, k, stride, pad)), np.float32)
    _load().oracle_maxpool2d(_p(x), *_i(N, C, H, W, k, stride, pad, 1 if relu else 0), _p(out))
    return out


def speedup_model(c, n_w):
    return float(_load().oracle_speedup_model(float(c), float(n_w)))
