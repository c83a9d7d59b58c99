"""CPU-side checks of the C-ABI library: it loads, exports every symbol the
header declares, and rejects bad arguments before touching the GPU."""
import ctypes
import os
import re

import pytest

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if f.endswith(".h"):
            src = open(os.path.join(inc, f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(xnor_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    lib = X.load()
    names = declared_functions()
    assert {"xnor_binarize_weights", "xnor_binactiv", "xnor_conv2d_forward"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTS) <= set(names)


def test_small_host_functions():
    assert X.xnor_version() >= 100
    assert X.xnor_words_per_pixel(1) == 1 and X.xnor_words_per_pixel(32) == 1
    assert X.xnor_words_per_pixel(33) == 2 and X.xnor_words_per_pixel(96) == 3
    assert X.xnor_out_extent(27, 5, 1, 2) == 27 and X.xnor_out_extent(56, 3, 2, 1) == 28
    assert X.xnor_out_extent(3, 7, 1, 1) == 0
    assert X.status_string(B.XNOR_OK) == "XNOR_OK"
    assert X.status_string(B.XNOR_ERR_TIMEOUT) == "XNOR_ERR_TIMEOUT"


def test_engine_switch():
    X.xnor_set_engine(B.XNOR_ENGINE_POPC)
    assert X.xnor_get_engine() == B.XNOR_ENGINE_POPC
    for e in (B.XNOR_ENGINE_UMMA, B.XNOR_ENGINE_UMMA_STREAM, B.XNOR_ENGINE_UMMA_SINGLE,
              B.XNOR_ENGINE_UMMA_PAIR, B.XNOR_ENGINE_UMMA_PAIR_STREAM, B.XNOR_ENGINE_AUTO):
        X.xnor_set_engine(e)
        assert X.xnor_get_engine() == e
    for bad in (-1, 7, 17):
        with pytest.raises(X.XnorError):
            X.xnor_set_engine(bad)
    assert X.xnor_get_engine() == B.XNOR_ENGINE_AUTO


def test_arguments_are_rejected_before_any_launch():
    """Null or misaligned pointers and impossible geometry return INVALID_ARG
    on the host; nothing is launched (this runs without a GPU)."""
    lib = X.load()
    p = ctypes.c_void_p(0x1000)        # aligned, never dereferenced on these paths
    odd = ctypes.c_void_p(0x1004)
    null = ctypes.c_void_p(0)
    inv = B.XNOR_ERR_INVALID_ARG
    assert lib.xnor_binarize_weights(null, 4, 4, 3, 3, p, p, null) == inv
    assert lib.xnor_binarize_weights(p, 4, 4, 3, 3, odd, p, null) == inv
    assert lib.xnor_binarize_weights(p, 0, 4, 3, 3, p, p, null) == inv
    assert lib.xnor_binarize_weights(p, 4, 1024, 20, 20, p, p, null) == B.XNOR_ERR_UNSUPPORTED
    d = X.make_desc(1, 8, 5, 5, 4, 3, 3, 1, 1)
    assert lib.xnor_binactiv(null, null, null, ctypes.byref(d), p, p, p, null) == inv
    assert lib.xnor_binactiv(p, p, null, ctypes.byref(d), p, p, p, null) == inv     # one BN vector only
    assert lib.xnor_binactiv(p, null, null, None, p, p, p, null) == inv
    assert lib.xnor_binactiv(p, null, null, ctypes.byref(d), p, null, p, null) == inv  # A is required
    for bad in (X.make_desc(0, 8, 5, 5, 4, 3, 3, 1, 1), X.make_desc(1, 8, 5, 5, 4, 3, 3, 0, 1),
                X.make_desc(1, 8, 5, 5, 4, 3, 3, 1, -1), X.make_desc(1, 8, 2, 2, 4, 7, 7, 1, 1)):
        assert lib.xnor_binactiv(p, null, null, ctypes.byref(bad), p, p, p, null) == inv
        assert lib.xnor_conv2d_forward(p, p, p, p, null, ctypes.byref(bad), p, null, null) == inv
    assert lib.xnor_conv2d_forward(p, p, p, p, null, ctypes.byref(d), null, null, null) == inv
    assert lib.xnor_conv2d_forward(p, p, p, p, odd, ctypes.byref(d), p, null, null) == inv
    nocout = X.make_desc(1, 8, 5, 5, 0, 3, 3, 1, 1)
    assert lib.xnor_conv2d_forward(p, p, p, p, null, ctypes.byref(nocout), p, null, null) == inv
    big = X.make_desc(1, 8, 32, 32, 4, 13, 13, 1, 6)
    assert lib.xnor_conv2d_forward(p, p, p, p, null, ctypes.byref(big), p, null, null) == \
        B.XNOR_ERR_UNSUPPORTED
    assert lib.xnor_shortcut_conv1x1(p, null, 1, 4, 4, 4, 4, 2, p, null) == inv
    assert lib.xnor_shortcut_conv1x1(p, p, 1, 4, 4, 4, 4, 0, p, null) == inv
    # option flags: unknown bits are an error
    badflag = X.make_desc(1, 8, 5, 5, 4, 3, 3, 1, 1, 8)
    assert lib.xnor_binactiv(p, null, null, ctypes.byref(badflag), p, p, p, null) == inv
    assert lib.xnor_conv2d_forward(p, p, p, p, null, ctypes.byref(badflag), p, null, null) == inv
    # shapes the BinActiv kernels do not cover are refused before any launch
    wide = X.make_desc(1, 4000, 5, 5, 4, 3, 3, 1, 1)
    assert lib.xnor_binactiv(p, p, p, ctypes.byref(wide), p, p, p, null) == B.XNOR_ERR_UNSUPPORTED
    many = X.make_desc(70000, 8, 2, 2, 4, 1, 1, 1, 0)
    assert lib.xnor_binactiv(p, null, null, ctypes.byref(many), p, p, p, null) == B.XNOR_ERR_UNSUPPORTED
    # k-bit calls: the number of bits is checked, then the same rules as the 1-bit calls
    for kb in (0, 8, -1):
        assert lib.xnor_binactiv_kbit(p, null, null, ctypes.byref(d), kb, p, p, p, null) == inv
        assert lib.xnor_conv2d_forward_kbit(p, kb, p, p, p, null, ctypes.byref(d), p, null, null) == inv
    assert lib.xnor_binactiv_kbit(p, null, null, ctypes.byref(d), 2, null, p, p, null) == inv
    assert lib.xnor_conv2d_forward_kbit(null, 2, p, p, p, null, ctypes.byref(d), p, null, null) == inv
    odd_planes = X.make_desc(1, 8, 5, 5, 4, 3, 3, 1, 1)          # 25 words per plane: not 16-byte aligned
    assert lib.xnor_conv2d_forward_kbit(p, 2, p, p, p, null, ctypes.byref(odd_planes), p, null, null) == \
        B.XNOR_ERR_UNSUPPORTED


def test_binding_refuses_host_tensors():
    import torch
    w = torch.zeros(4, 4, 3, 3)
    wp, al = torch.zeros(4, 3, 3, 1, dtype=torch.int32), torch.zeros(4)
    with pytest.raises(ValueError):
        X.xnor_binarize_weights(w, wp, al, stream=0)
