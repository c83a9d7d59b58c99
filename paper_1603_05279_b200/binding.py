"""ctypes binding of libxnor.so: argument marshalling only.

Each function has the name and argument order of the C entry point it
forwards to (see include/xnor.h) and takes torch CUDA tensors where the C call
takes device pointers.  Nothing here computes: a missing or unloadable library
raises, there is no fallback.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# XNOR_LIB selects another build of the same library in this directory (the checking build,
# libxnor_check.so); nothing else is ever loaded.
LIB_PATH = os.path.join(_HERE, os.path.basename(os.environ.get("XNOR_LIB", "libxnor.so")))

XNOR_OK = 0
XNOR_ERR_INVALID_ARG = 1
XNOR_ERR_UNSUPPORTED = 2
XNOR_ERR_CUDA = 3
XNOR_ERR_TIMEOUT = 4
XNOR_ERR_BOUNDS = 5

XNOR_FLAG_RELU = 1
XNOR_FLAG_K_VALID_TAPS = 2

XNOR_ENGINE_AUTO = 0
XNOR_ENGINE_POPC = 1
XNOR_ENGINE_UMMA = 2
XNOR_ENGINE_UMMA_STREAM = 3
XNOR_ENGINE_UMMA_SINGLE = 4
XNOR_ENGINE_UMMA_PAIR = 5
XNOR_ENGINE_UMMA_PAIR_STREAM = 6

EXPORTS = [
    "xnor_version", "xnor_built_with_bounds_check", "xnor_status_string", "xnor_words_per_pixel", "xnor_out_extent",
    "xnor_binarize_weights", "xnor_binactiv", "xnor_binactiv_static", "xnor_conv2d_forward", "xnor_shortcut_conv1x1",
    "xnor_set_engine", "xnor_get_engine", "xnor_check_device", "xnor_selftest_wait_timeout",
    "xnor_maxpool2d", "xnor_binactiv_launches", "xnor_binactiv_kbit_launches", "xnor_conv2d_binactiv_parts", "xnor_conv2d_forward_binactiv", "xnor_binactiv_finish",
    "xnor_binactiv_kbit", "xnor_conv2d_forward_kbit",
    "xnor_bwn_input_elems", "xnor_bwn_prepare_input", "xnor_bwn_conv2d_forward",
    "xnor_bgrad_stream_elems", "xnor_binarize_weights_transposed", "xnor_binary_gradient_backward", "xnor_measure_peaks",
]


class xnor_conv_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("N", "C_in", "H", "W", "C_out", "k_h", "k_w", "stride", "pad", "flags")]


class XnorError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s returned %s" % (where, status_string(status)))


_lib = None


def load():
    """Load libxnor.so (built in-tree by paper_1603_05279_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("libxnor.so is not built: run `python -m paper_1603_05279_b200.build` "
                          "(needs nvcc); there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.xnor_version.restype = ci
    lib.xnor_built_with_bounds_check.restype = ci
    lib.xnor_status_string.restype = ctypes.c_char_p
    lib.xnor_status_string.argtypes = [ci]
    lib.xnor_words_per_pixel.restype = ctypes.c_size_t
    lib.xnor_words_per_pixel.argtypes = [ci]
    lib.xnor_out_extent.restype = ci
    lib.xnor_out_extent.argtypes = [ci] * 4
    lib.xnor_binarize_weights.restype = ci
    lib.xnor_binarize_weights.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp]
    lib.xnor_binactiv.restype = ci
    lib.xnor_binactiv.argtypes = [vp, vp, vp, ctypes.POINTER(xnor_conv_desc), vp, vp, vp, vp]
    lib.xnor_binactiv_static.restype = ci
    lib.xnor_binactiv_static.argtypes = [vp, vp, vp, ctypes.POINTER(xnor_conv_desc), vp, vp, vp]
    lib.xnor_conv2d_forward.restype = ci
    lib.xnor_conv2d_forward.argtypes = [vp, vp, vp, vp, vp, ctypes.POINTER(xnor_conv_desc),
                                        vp, vp, vp]
    lib.xnor_shortcut_conv1x1.restype = ci
    lib.xnor_shortcut_conv1x1.argtypes = [vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
    lib.xnor_set_engine.restype = ci
    lib.xnor_set_engine.argtypes = [ci]
    lib.xnor_get_engine.restype = ci
    lib.xnor_check_device.restype = ci
    lib.xnor_check_device.argtypes = [vp]
    lib.xnor_conv2d_binactiv_parts.restype = ci
    lib.xnor_binactiv_kbit_launches.restype = ci
    lib.xnor_binactiv_kbit_launches.argtypes = [ctypes.POINTER(xnor_conv_desc), ci, ci]
    lib.xnor_binactiv_launches.restype = ci
    lib.xnor_binactiv_launches.argtypes = [ctypes.POINTER(xnor_conv_desc), ci]
    lib.xnor_conv2d_binactiv_parts.argtypes = [ctypes.POINTER(xnor_conv_desc)]
    lib.xnor_conv2d_forward_binactiv.restype = ci
    lib.xnor_conv2d_forward_binactiv.argtypes = [vp, vp, vp, vp, vp, ctypes.POINTER(xnor_conv_desc), vp,
                                                 vp, vp, vp, vp, vp]
    lib.xnor_binactiv_finish.restype = ci
    lib.xnor_binactiv_finish.argtypes = [vp, ci, ctypes.POINTER(xnor_conv_desc), vp, vp, vp]
    lib.xnor_maxpool2d.restype = ci
    lib.xnor_maxpool2d.argtypes = [vp, ci, ci, ci, ci, ci, ci, ci, ci, vp, vp]
    lib.xnor_selftest_wait_timeout.restype = ci
    lib.xnor_selftest_wait_timeout.argtypes = [vp]
    lib.xnor_binactiv_kbit.restype = ci
    lib.xnor_binactiv_kbit.argtypes = [vp, vp, vp, ctypes.POINTER(xnor_conv_desc), ci, vp, vp, vp, vp]
    lib.xnor_conv2d_forward_kbit.restype = ci
    lib.xnor_conv2d_forward_kbit.argtypes = [vp, ci, vp, vp, vp, vp, ctypes.POINTER(xnor_conv_desc),
                                             vp, vp, vp]
    lib.xnor_bwn_input_elems.restype = ctypes.c_size_t
    lib.xnor_bwn_input_elems.argtypes = [ctypes.POINTER(xnor_conv_desc)]
    lib.xnor_bwn_prepare_input.restype = ci
    lib.xnor_bwn_prepare_input.argtypes = [vp, vp, vp, ctypes.POINTER(xnor_conv_desc), vp, vp]
    lib.xnor_bwn_conv2d_forward.restype = ci
    lib.xnor_bwn_conv2d_forward.argtypes = [vp, vp, vp, vp, ctypes.POINTER(xnor_conv_desc), vp, vp]
    lib.xnor_bgrad_stream_elems.restype = ctypes.c_size_t
    lib.xnor_bgrad_stream_elems.argtypes = [ctypes.POINTER(xnor_conv_desc)]
    lib.xnor_binarize_weights_transposed.restype = ci
    lib.xnor_binarize_weights_transposed.argtypes = [vp, ci, ci, ci, ci, vp, vp]
    lib.xnor_binary_gradient_backward.restype = ci
    lib.xnor_binary_gradient_backward.argtypes = [vp, vp, vp, ctypes.POINTER(xnor_conv_desc), vp, vp, vp, vp]
    lib.xnor_measure_peaks.restype = ci
    lib.xnor_measure_peaks.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), vp]
    _lib = lib
    return lib


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("libxnor takes device pointers: tensor is on %s" % t.device)
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError("expected %s, got %s" % (dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(status, where):
    if status != XNOR_OK:
        raise XnorError(status, where)


def make_desc(N, C_in, H, W, C_out, k_h, k_w, stride, pad, flags=0):
    return xnor_conv_desc(N, C_in, H, W, C_out, k_h, k_w, stride, pad, flags)


def desc_of(s):
    """xnor_conv_desc of a workloads.ConvShape."""
    return xnor_conv_desc(s.N, s.C_in, s.H, s.W, s.C_out, s.k, s.k, s.stride, s.pad, 0)


def xnor_version():
    return int(load().xnor_version())


def xnor_built_with_bounds_check():
    return int(load().xnor_built_with_bounds_check())


def status_string(status):
    return load().xnor_status_string(int(status)).decode()


def xnor_words_per_pixel(C_in):
    return int(load().xnor_words_per_pixel(int(C_in)))


def xnor_out_extent(n, k, stride, pad):
    return int(load().xnor_out_extent(int(n), int(k), int(stride), int(pad)))


def xnor_set_engine(engine):
    _check(load().xnor_set_engine(int(engine)), "xnor_set_engine")


def xnor_get_engine():
    return int(load().xnor_get_engine())


def xnor_check_device(stream=None):
    """Synchronises the stream and raises XnorError if a device-side wait expired."""
    _check(load().xnor_check_device(_stream(stream)), "xnor_check_device")


def xnor_binactiv_launches(d, has_bn=False):
    """Kernels xnor_binactiv launches for this shape (1 or 2; 0 = refused shape)."""
    return int(load().xnor_binactiv_launches(ctypes.byref(d), int(bool(has_bn))))


def xnor_binactiv_kbit_launches(d, kbits, has_bn=False):
    """Kernels xnor_binactiv_kbit launches for this shape (1 or 2; 0 = bad arguments)."""
    return int(load().xnor_binactiv_kbit_launches(ctypes.byref(d), int(kbits), int(bool(has_bn))))


def xnor_conv2d_binactiv_parts(d):
    """Partial planes the fused call writes for this shape (0: not covered)."""
    return int(load().xnor_conv2d_binactiv_parts(ctypes.byref(d)))


def xnor_conv2d_forward_binactiv(x_packed, w_packed, alpha, K, residual, d, out, next_scale,
                                 next_shift, x_packed_next, A_parts, stream=None):
    _check(load().xnor_conv2d_forward_binactiv(
        _ptr(x_packed, torch.int32), _ptr(w_packed, torch.int32), _ptr(alpha, torch.float32),
        _ptr(K, torch.float32), _ptr(residual, torch.float32) if residual is not None else None,
        ctypes.byref(d), _ptr(out, torch.float32) if out is not None else None,
        _ptr(next_scale, torch.float32) if next_scale is not None else None,
        _ptr(next_shift, torch.float32) if next_shift is not None else None,
        _ptr(x_packed_next, torch.int32), _ptr(A_parts, torch.float32), _stream(stream)),
        "xnor_conv2d_forward_binactiv")


def xnor_binactiv_finish(A_parts, parts, d_next, A, K, stream=None):
    _check(load().xnor_binactiv_finish(_ptr(A_parts, torch.float32), int(parts), ctypes.byref(d_next),
                                       _ptr(A, torch.float32), _ptr(K, torch.float32), _stream(stream)),
           "xnor_binactiv_finish")


def xnor_maxpool2d(x, k, stride, pad, relu, out, stream=None):
    N, C, H, W = x.shape
    _check(load().xnor_maxpool2d(_ptr(x, torch.float32), N, C, H, W, int(k), int(stride), int(pad),
                                 1 if relu else 0, _ptr(out, torch.float32), _stream(stream)),
           "xnor_maxpool2d")


def xnor_selftest_wait_timeout(stream=None):
    """Launches the one-warp kernel whose bounded wait expires (see the header)."""
    _check(load().xnor_selftest_wait_timeout(_stream(stream)), "xnor_selftest_wait_timeout")


def xnor_binarize_weights(w, w_packed, alpha, stream=None):
    C_out, C_in, k_h, k_w = w.shape
    _check(load().xnor_binarize_weights(_ptr(w, torch.float32), C_out, C_in, k_h, k_w,
                                        _ptr(w_packed, torch.int32), _ptr(alpha, torch.float32),
                                        _stream(stream)), "xnor_binarize_weights")


def xnor_binactiv(x, bn_scale, bn_shift, d, x_packed, A, K, stream=None):
    _check(load().xnor_binactiv(_ptr(x, torch.float32), _ptr(bn_scale, torch.float32),
                                _ptr(bn_shift, torch.float32), ctypes.byref(d),
                                _ptr(x_packed, torch.int32), _ptr(A, torch.float32),
                                _ptr(K, torch.float32), _stream(stream)), "xnor_binactiv")


def xnor_binactiv_kbit(x, bn_scale, bn_shift, d, kbits, x_planes, A, K, stream=None):
    _check(load().xnor_binactiv_kbit(_ptr(x, torch.float32), _ptr(bn_scale, torch.float32),
                                     _ptr(bn_shift, torch.float32), ctypes.byref(d), int(kbits),
                                     _ptr(x_planes, torch.int32), _ptr(A, torch.float32),
                                     _ptr(K, torch.float32), _stream(stream)), "xnor_binactiv_kbit")


def xnor_conv2d_forward_kbit(x_planes, kbits, w_packed, alpha, K, residual, d, out, acc_out=None,
                             stream=None):
    _check(load().xnor_conv2d_forward_kbit(_ptr(x_planes, torch.int32), int(kbits),
                                           _ptr(w_packed, torch.int32), _ptr(alpha, torch.float32),
                                           _ptr(K, torch.float32), _ptr(residual, torch.float32),
                                           ctypes.byref(d), _ptr(out, torch.float32),
                                           _ptr(acc_out, torch.int32), _stream(stream)),
           "xnor_conv2d_forward_kbit")


def xnor_measure_peaks(stream=None):
    """(1-bit MACs per clock per SM on the tensor pipe, popc per clock per SM), measured now."""
    a, b = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(load().xnor_measure_peaks(ctypes.byref(a), ctypes.byref(b), _stream(stream)), "xnor_measure_peaks")
    return a.value, b.value


def xnor_bwn_input_elems(d):
    return int(load().xnor_bwn_input_elems(ctypes.byref(d)))


def xnor_bwn_prepare_input(x, bn_scale, bn_shift, d, x_stream, stream=None):
    _check(load().xnor_bwn_prepare_input(_ptr(x, torch.float32), _ptr(bn_scale, torch.float32),
                                         _ptr(bn_shift, torch.float32), ctypes.byref(d),
                                         _ptr(x_stream, torch.bfloat16), _stream(stream)),
           "xnor_bwn_prepare_input")


def xnor_bwn_conv2d_forward(x_stream, w_packed, alpha, residual, d, out, stream=None):
    _check(load().xnor_bwn_conv2d_forward(_ptr(x_stream, torch.bfloat16), _ptr(w_packed, torch.int32),
                                          _ptr(alpha, torch.float32), _ptr(residual, torch.float32),
                                          ctypes.byref(d), _ptr(out, torch.float32), _stream(stream)),
           "xnor_bwn_conv2d_forward")


def xnor_bgrad_stream_elems(d):
    return int(load().xnor_bgrad_stream_elems(ctypes.byref(d)))


def xnor_binarize_weights_transposed(w, wT_packed, stream=None):
    """w fp32 [C_out][C_in][k_h][k_w] -> sign bits for the backward convolution (alloc_weights_transposed)."""
    Co, C, kh, kw = w.shape
    _check(load().xnor_binarize_weights_transposed(_ptr(w, torch.float32), Co, C, kh, kw,
                                                   _ptr(wT_packed, torch.int32), _stream(stream)),
           "xnor_binarize_weights_transposed")


def xnor_binary_gradient_backward(g, wT_packed, alpha, d, gmax, g_stream, grad_in, stream=None):
    _check(load().xnor_binary_gradient_backward(_ptr(g, torch.float32), _ptr(wT_packed, torch.int32),
                                                _ptr(alpha, torch.float32), ctypes.byref(d),
                                                _ptr(gmax, torch.float32), _ptr(g_stream, torch.bfloat16),
                                                _ptr(grad_in, torch.float32), _stream(stream)),
           "xnor_binary_gradient_backward")


def alloc_weights_transposed(C_out, C_in, k_h, k_w, device="cuda"):
    """Packed sign words [P'][C_in][2] of the backward convolution."""
    pairs = (k_h * k_w * ((C_out + 31) // 32) + 1) // 2
    return torch.empty((pairs, C_in, 2), dtype=torch.int32, device=device)


def alloc_bgrad(d, device="cuda"):
    """(gmax [N], g_stream scratch, grad_in [N][C_in][H][W]) for xnor_binary_gradient_backward."""
    return (torch.empty((d.N,), dtype=torch.float32, device=device),
            torch.empty((xnor_bgrad_stream_elems(d),), dtype=torch.bfloat16, device=device),
            torch.empty((d.N, d.C_in, d.H, d.W), dtype=torch.float32, device=device))


def alloc_bwn_input(d, device="cuda"):
    return torch.empty((xnor_bwn_input_elems(d),), dtype=torch.bfloat16, device=device)


BINACTIV_STATIC_MAX_PIXELS = 1 << 20


def xnor_binactiv_static(x, bn_scale, bn_shift, d, x_packed, K, stream=None):
    """xnor_binactiv for callers that cannot supply the A buffer: A lives in a fixed
    4 MiB array inside the library (at most BINACTIV_STATIC_MAX_PIXELS pixels per call)."""
    _check(load().xnor_binactiv_static(_ptr(x, torch.float32), _ptr(bn_scale, torch.float32),
                                       _ptr(bn_shift, torch.float32), ctypes.byref(d),
                                       _ptr(x_packed, torch.int32), _ptr(K, torch.float32),
                                       _stream(stream)), "xnor_binactiv_static")


def xnor_conv2d_forward(x_packed, w_packed, alpha, K, residual, d, out, acc_out=None, stream=None):
    _check(load().xnor_conv2d_forward(_ptr(x_packed, torch.int32), _ptr(w_packed, torch.int32),
                                      _ptr(alpha, torch.float32), _ptr(K, torch.float32),
                                      _ptr(residual, torch.float32), ctypes.byref(d),
                                      _ptr(out, torch.float32), _ptr(acc_out, torch.int32),
                                      _stream(stream)), "xnor_conv2d_forward")


def xnor_shortcut_conv1x1(x, w, stride, out, stream=None):
    N, C_in, H, W = x.shape
    C_out = w.shape[0]
    _check(load().xnor_shortcut_conv1x1(_ptr(x, torch.float32), _ptr(w, torch.float32), N, C_in,
                                        H, W, C_out, int(stride), _ptr(out, torch.float32),
                                        _stream(stream)), "xnor_shortcut_conv1x1")


# ---- buffer helpers (allocation only; torch owns the memory) -------------------------------
def alloc_weights(C_out, C_in, k_h, k_w, device="cuda"):
    Cw = (C_in + 31) // 32
    pairs = (k_h * k_w * Cw + 1) // 2          # word-pair-major layout, see include/xnor.h
    return (torch.empty((pairs, C_out, 2), dtype=torch.int32, device=device),
            torch.empty((C_out,), dtype=torch.float32, device=device))


def alloc_binactiv(d, device="cuda"):
    Cw = (d.C_in + 31) // 32
    Ho = (d.H + 2 * d.pad - d.k_h) // d.stride + 1
    Wo = (d.W + 2 * d.pad - d.k_w) // d.stride + 1
    return (torch.empty((d.N, d.H, d.W, Cw), dtype=torch.int32, device=device),
            torch.empty((d.N, d.H, d.W), dtype=torch.float32, device=device),
            torch.empty((d.N, Ho, Wo), dtype=torch.float32, device=device))


def alloc_out(d, dtype=torch.float32, device="cuda"):
    Ho = (d.H + 2 * d.pad - d.k_h) // d.stride + 1
    Wo = (d.W + 2 * d.pad - d.k_w) // d.stride + 1
    return torch.empty((d.N, d.C_out, Ho, Wo), dtype=dtype, device=device)
