"""Device buffers and launch sequence of one XNOR block per layer.

Marshalling only: it owns torch tensors and calls the C-ABI entry points in
the paper's order (weight binarisation, then BN -> BinActiv -> BinConv).
"""
import torch

from . import binding as B
from . import workloads as wl


class LayerBuffers:
    """All device tensors of one layer; inputs are filled by the caller."""

    def __init__(self, shape, device="cuda", with_acc=False, with_bn=True):
        s = shape
        self.shape = s
        self.desc = B.desc_of(s)
        self.x = torch.empty((s.N, s.C_in, s.H, s.W), dtype=torch.float32, device=device)
        self.w = torch.empty((s.C_out, s.C_in, s.k, s.k), dtype=torch.float32, device=device)
        self.bn_scale = torch.ones((s.C_in,), dtype=torch.float32, device=device) if with_bn else None
        self.bn_shift = torch.zeros((s.C_in,), dtype=torch.float32, device=device) if with_bn else None
        self.w_packed, self.alpha = B.alloc_weights(s.C_out, s.C_in, s.k, s.k, device)
        self.x_packed, self.A, self.K = B.alloc_binactiv(self.desc, device)
        self.out = B.alloc_out(self.desc, device=device)
        self.acc = B.alloc_out(self.desc, torch.int32, device) if with_acc else None
        self.residual = None

    def binarize_weights(self, stream=None):
        B.xnor_binarize_weights(self.w, self.w_packed, self.alpha, stream)

    def binactiv(self, stream=None):
        B.xnor_binactiv(self.x, self.bn_scale, self.bn_shift, self.desc, self.x_packed, self.A,
                        self.K, stream)

    def conv(self, stream=None):
        B.xnor_conv2d_forward(self.x_packed, self.w_packed, self.alpha, self.K, self.residual,
                              self.desc, self.out, self.acc, stream)

    def forward(self, stream=None, with_weights=True):
        if with_weights:
            self.binarize_weights(stream)
        self.binactiv(stream)
        self.conv(stream)

    # algorithmic bytes, as the roofline of each kernel counts them
    def binactiv_bytes(self):
        s = self.shape
        ho, wo = wl.out_hw(s)
        cw = (s.C_in + 31) // 32
        px = s.N * s.H * s.W
        return 4 * (px * s.C_in + px * cw + 2 * px + s.N * ho * wo)

    def conv_bytes(self):
        s = self.shape
        ho, wo = wl.out_hw(s)
        cw = (s.C_in + 31) // 32
        m = s.N * ho * wo
        return 4 * (s.N * s.H * s.W * cw + s.C_out * s.k * s.k * cw + m + s.C_out + m * s.C_out)

    def weight_bytes(self):
        s = self.shape
        return 4 * s.C_out * s.C_in * s.k * s.k


# kernels launched by one forward(): binarize 1, binactiv 2 (pack, box filter), conv 1
LAUNCHES_PER_LAYER = 4
