"""Helpers shared by the GPU parity tests (no arithmetic of the method)."""
import numpy as np
import torch

REL_TOL = 1e-5   # fp32 outputs: max |gpu - oracle| <= REL_TOL * max |oracle|


def unpack_bits(words, C):
    """u32/i32 words [..., Cw] -> +-1 int8 [..., C]; also checks the tail bits are 0."""
    w = np.ascontiguousarray(words).view(np.uint32)
    Cw = w.shape[-1]
    bits = ((w[..., :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(*w.shape[:-1], Cw * 32)
    assert not bits[..., C:].any(), "tail bits of the last word must be 0"
    return np.where(bits[..., :C] == 1, 1, -1).astype(np.int8)


def unpack_activations(x_packed, C):
    """[N][H][W][Cw] words -> +-1 [N][C][H][W]."""
    return np.ascontiguousarray(unpack_bits(x_packed, C).transpose(0, 3, 1, 2))


def unpack_weights(w_packed, C, kh, kw):
    """Word-pair-major words [pairs][Co][2] -> +-1 [Co][C][kh][kw].  Word f = (ky*kw + kx)*Cw + cw
    of filter co is element [f // 2][co][f % 2]; an odd word count is padded with a 0 word."""
    w = np.ascontiguousarray(w_packed)
    pairs, Co, _ = w.shape
    Cw = (C + 31) // 32
    nwords = kh * kw * Cw
    assert pairs == (nwords + 1) // 2
    flat = w.transpose(1, 0, 2).reshape(Co, pairs * 2)
    assert not flat[:, nwords:].any(), "padding word must be 0"
    words = np.ascontiguousarray(flat[:, :nwords]).reshape(Co, kh, kw, Cw)
    return np.ascontiguousarray(unpack_bits(words, C).transpose(0, 3, 1, 2))


def assert_close(gpu, ref, what, rel=REL_TOL):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (what, gpu.shape, ref.shape)
    scale = np.abs(ref).max() if ref.size else 0.0
    err = np.abs(gpu - ref).max() if ref.size else 0.0
    assert err <= rel * scale + 1e-30, "%s: max abs err %.3e > %.1e * max|ref| (%.3e)" % (
        what, err, rel, scale)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()


# ---- guard words around output buffers ------------------------------------------------------
# A kernel that writes outside a buffer it was given usually lands in a neighbouring
# allocation and goes unnoticed.  Outputs of the parity tests are therefore carved out of a
# larger allocation whose head and tail hold a known pattern, checked after the calls.
GUARD = 64                      # elements on each side (a multiple of 16 bytes for 2- and 4-byte types)
_PATTERN = {torch.float32: -7.25e30, torch.int32: -0x5A5A5A5B, torch.bfloat16: -7.25e30}


class Guarded:
    """A CUDA tensor of `shape` with GUARD pattern elements before and after it."""

    def __init__(self, shape, dtype=torch.float32, fill=None):
        n = int(np.prod(shape)) if len(shape) else 1
        self.raw = torch.empty(n + 2 * GUARD, dtype=dtype, device="cuda")
        self.pattern = _PATTERN[dtype]
        self.raw.fill_(self.pattern)
        self.t = self.raw[GUARD:GUARD + n].view(*shape)
        if fill is not None:
            self.t.fill_(fill)
        assert self.t.data_ptr() % 16 == 0

    def check(self, what=""):
        head, tail = self.raw[:GUARD], self.raw[-GUARD:]
        ok = bool((head == self.pattern).all()) and bool((tail == self.pattern).all())
        assert ok, "write outside the buffer: %s" % what


class GuardSet:
    """Allocates guarded outputs by name and checks them all at once."""

    def __init__(self):
        self.items = {}

    def new(self, name, shape, dtype=torch.float32, fill=None):
        g = Guarded(tuple(shape), dtype, fill)
        self.items[name] = g
        return g.t

    def like(self, name, t):
        return self.new(name, t.shape, t.dtype)

    def check(self):
        torch.cuda.synchronize()
        for name, g in self.items.items():
            g.check(name)
