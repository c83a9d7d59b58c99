"""Device buffers and launch sequence of one XNOR block per layer.

Marshalling only: it owns torch tensors and calls the C-ABI entry points in
the paper's order (weight binarisation, then BN -> BinActiv -> BinConv).
"""
import torch

from . import binding as B
from . import workloads as wl


class LayerBuffers:
    """All device tensors of one layer; inputs are filled by the caller."""

    def __init__(self, shape, device="cuda", with_acc=False, with_bn=True, variant="xnor", kbits=2):
        """variant: "xnor" (the block of Eq. 11), "bwn" (real inputs, binary weights, Eq. 1),
        "kbit" (q_k activations with `kbits` bits in place of sign) or "bgrad" (the layer's backward
        convolution with a binarised gradient: x is then the gradient at the layer's output,
        [N][C_out][H_out][W_out], and out the gradient at its input, [N][C_in][H][W])."""
        s = shape
        self.variant, self.kbits = variant, kbits
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
        if variant == "bwn":
            self.x_stream = B.alloc_bwn_input(self.desc, device)
        elif variant == "kbit":
            self.x_planes = torch.empty((kbits,) + tuple(self.x_packed.shape), dtype=torch.int32,
                                        device=device)
        elif variant == "bgrad":
            self.x = torch.empty(tuple(self.out.shape), dtype=torch.float32, device=device)
            self.wT_packed = B.alloc_weights_transposed(s.C_out, s.C_in, s.k, s.k, device)
            self.gmax, self.g_stream, self.out = B.alloc_bgrad(self.desc, device)

    def binarize_weights(self, stream=None):
        B.xnor_binarize_weights(self.w, self.w_packed, self.alpha, stream)
        if self.variant == "bgrad":
            B.xnor_binarize_weights_transposed(self.w, self.wT_packed, stream)

    def binactiv(self, stream=None):
        if self.variant == "bgrad":
            return                   # the gradient is scaled and laid out inside the backward call
        if self.variant == "bwn":
            B.xnor_bwn_prepare_input(self.x, self.bn_scale, self.bn_shift, self.desc, self.x_stream, stream)
        elif self.variant == "kbit":
            B.xnor_binactiv_kbit(self.x, self.bn_scale, self.bn_shift, self.desc, self.kbits,
                                 self.x_planes, self.A, self.K, stream)
        else:
            B.xnor_binactiv(self.x, self.bn_scale, self.bn_shift, self.desc, self.x_packed, self.A,
                            self.K, stream)

    def conv(self, stream=None):
        if self.variant == "bgrad":
            B.xnor_binary_gradient_backward(self.x, self.wT_packed, self.alpha, self.desc, self.gmax,
                                            self.g_stream, self.out, stream)
        elif self.variant == "bwn":
            B.xnor_bwn_conv2d_forward(self.x_stream, self.w_packed, self.alpha, self.residual,
                                      self.desc, self.out, stream)
        elif self.variant == "kbit":
            B.xnor_conv2d_forward_kbit(self.x_planes, self.kbits, self.w_packed, self.alpha, self.K,
                                       self.residual, self.desc, self.out, self.acc, stream)
        else:
            B.xnor_conv2d_forward(self.x_packed, self.w_packed, self.alpha, self.K, self.residual,
                                  self.desc, self.out, self.acc, stream)

    def forward(self, stream=None, with_weights=True):
        if with_weights:
            self.binarize_weights(stream)
        self.binactiv(stream)
        self.conv(stream)

    # algorithmic bytes, as the roofline of each kernel counts them
    def binactiv_launches(self):
        if self.variant == "bgrad":
            return 0
        if self.variant == "bwn":
            return 1
        if self.variant == "kbit":
            return B.xnor_binactiv_kbit_launches(self.desc, self.kbits, self.bn_scale is not None)
        return B.xnor_binactiv_launches(self.desc, self.bn_scale is not None)

    def launches(self):
        """Kernels one forward() launches: binarize 1, BinActiv 1 or 2 (pack + A, box filter; one
        kernel where a block streams whole images), BinConv 1 (k-bit: one per plane)."""
        if self.variant == "bgrad":
            return 2 + 3             # two weight packings; maximum, gradient stream, convolution
        conv = self.kbits if self.variant == "kbit" else 1
        return 1 + self.binactiv_launches() + conv

    def binactiv_bytes(self):
        if self.variant == "bgrad":
            return 0
        s = self.shape
        ho, wo = wl.out_hw(s)
        cw = (s.C_in + 31) // 32
        px = s.N * s.H * s.W
        # A is written once and, where K comes from a second kernel, read once
        a_passes = 2 if self.binactiv_launches() == 2 else 1
        return 4 * (px * s.C_in + px * cw + a_passes * px + s.N * ho * wo)

    def conv_bytes(self):
        s = self.shape
        ho, wo = wl.out_hw(s)
        cw = (s.C_in + 31) // 32
        m = s.N * ho * wo
        return 4 * (s.N * s.H * s.W * cw + s.C_out * s.k * s.k * cw + m + s.C_out + m * s.C_out)

    def weight_bytes(self):
        s = self.shape
        return 4 * s.C_out * s.C_in * s.k * s.k




class ChainRunner:
    """The 16 binary 3x3 layers of the ResNet-18 variant (Section 4.2) as 8 basic blocks:

        y1 = BinConv1(BinActiv(BN1(x)))
        y2 = BinConv2(BinActiv(BN2(y1))) + shortcut(x)

    shortcut = identity, or the fp32 1x1 stride-2 projection where the shape
    changes.  Launch sequence and buffers only; every step is a library call.
    BatchNorm enters as per-channel (scale, shift) vectors that the caller sets
    (see `calibrate`).
    """

    def __init__(self, N, device="cuda", keep_acc=False):
        self.N = N
        self.shapes = wl.chain_shapes(N)
        self.device = device
        s0 = self.shapes[0]
        self.x0 = torch.empty((N, s0.C_in, s0.H, s0.W), dtype=torch.float32, device=device)
        self.layers = []
        for s in self.shapes:
            d = B.desc_of(s)
            L = {"shape": s, "desc": d}
            L["w"] = torch.empty((s.C_out, s.C_in, s.k, s.k), dtype=torch.float32, device=device)
            L["w_packed"], L["alpha"] = B.alloc_weights(s.C_out, s.C_in, s.k, s.k, device)
            L["x_packed"], L["A"], L["K"] = B.alloc_binactiv(d, device)
            L["scale"] = torch.ones((s.C_in,), dtype=torch.float32, device=device)
            L["shift"] = torch.zeros((s.C_in,), dtype=torch.float32, device=device)
            L["out"] = B.alloc_out(d, device=device)
            L["acc"] = B.alloc_out(d, torch.int32, device) if keep_acc else None
            self.layers.append(L)
        # projection shortcuts: one per block whose first layer has stride 2
        self.proj = {}
        for i in range(0, len(self.shapes), 2):
            s = self.shapes[i]
            if s.stride != 1 or s.C_in != s.C_out:
                ho, wo = wl.out_hw(s)
                self.proj[i] = {
                    "w": torch.empty((s.C_out, s.C_in), dtype=torch.float32, device=device),
                    "out": torch.empty((N, s.C_out, ho, wo), dtype=torch.float32, device=device)}

    def layer_input(self, i):
        return self.x0 if i == 0 else self.layers[i - 1]["out"]

    def binarize_weights(self, stream=None):
        for L in self.layers:
            B.xnor_binarize_weights(L["w"], L["w_packed"], L["alpha"], stream)

    def run_layer(self, i, stream=None):
        """BN -> BinActiv -> BinConv of layer i (plus the block's shortcut on odd i)."""
        L = self.layers[i]
        x = self.layer_input(i)
        B.xnor_binactiv(x, L["scale"], L["shift"], L["desc"], L["x_packed"], L["A"], L["K"], stream)
        residual = None
        if i % 2 == 1:
            b0 = i - 1
            if b0 in self.proj:
                P = self.proj[b0]
                B.xnor_shortcut_conv1x1(self.layer_input(b0), P["w"], self.shapes[b0].stride,
                                        P["out"], stream)
                residual = P["out"]
            else:
                residual = self.layer_input(b0)
        B.xnor_conv2d_forward(L["x_packed"], L["w_packed"], L["alpha"], L["K"], residual,
                              L["desc"], L["out"], L["acc"], stream)
        return residual

    def forward(self, stream=None):
        for i in range(len(self.layers)):
            self.run_layer(i, stream)
        return self.layers[-1]["out"]

    def prepare_fused(self):
        """Buffers of the fused forward: for every layer but the last, the partial |y| planes
        its fused epilogue writes (0 parts: the shape is not covered and the layer runs the two
        plain calls).  The engine in force now must be the one used by forward_fused."""
        self.fused_parts = []
        for i, L in enumerate(self.layers[:-1]):
            parts = B.xnor_conv2d_binactiv_parts(L["desc"])
            self.fused_parts.append(parts)
            ho, wo = wl.out_hw(L["shape"])
            L["A_parts"] = torch.empty((max(parts, 1), self.N, ho, wo), dtype=torch.float32,
                                       device=self.device)
        self.fused_parts.append(0)

    def forward_fused(self, stream=None):
        """The same chain with each BinConv emitting the next layer's BinActiv from its epilogue.
        The output of a block's first convolution is consumed only by that BinActiv, so it is
        never written as fp32; a block's output is (it is the next block's shortcut input)."""
        n = len(self.layers)
        L0 = self.layers[0]
        B.xnor_binactiv(self.x0, L0["scale"], L0["shift"], L0["desc"], L0["x_packed"], L0["A"], L0["K"],
                        stream)
        for i, L in enumerate(self.layers):
            residual = None
            if i % 2 == 1:
                b0 = i - 1
                if b0 in self.proj:
                    P = self.proj[b0]
                    B.xnor_shortcut_conv1x1(self.layer_input(b0), P["w"], self.shapes[b0].stride,
                                            P["out"], stream)
                    residual = P["out"]
                else:
                    residual = self.layer_input(b0)
            parts = self.fused_parts[i]
            if parts > 0:
                nxt = self.layers[i + 1]
                out = L["out"] if i % 2 == 1 else None
                B.xnor_conv2d_forward_binactiv(L["x_packed"], L["w_packed"], L["alpha"], L["K"],
                                               residual, L["desc"], out, nxt["scale"], nxt["shift"],
                                               nxt["x_packed"], L["A_parts"], stream)
                B.xnor_binactiv_finish(L["A_parts"], parts, nxt["desc"], nxt["A"], nxt["K"], stream)
            else:
                B.xnor_conv2d_forward(L["x_packed"], L["w_packed"], L["alpha"], L["K"], residual,
                                      L["desc"], L["out"], None, stream)
                if i + 1 < n:
                    nxt = self.layers[i + 1]
                    B.xnor_binactiv(L["out"], nxt["scale"], nxt["shift"], nxt["desc"],
                                    nxt["x_packed"], nxt["A"], nxt["K"], stream)
        return self.layers[-1]["out"]

    def calibrate(self, eps=1e-5, stream=None):
        """Sets every BatchNorm to the statistics of its own input on the current batch
        (biased variance, gamma = 1, beta = 0), layer by layer.  Set-up, not the timed path:
        the statistics are plain torch reductions; the folded (scale, shift) vectors are what
        the library (and any checker) receives."""
        for i, L in enumerate(self.layers):
            x = self.layer_input(i).double()
            mean = x.mean(dim=(0, 2, 3))
            var = x.var(dim=(0, 2, 3), unbiased=False)
            scale = 1.0 / torch.sqrt(var + eps)
            L["scale"].copy_(scale.float())
            L["shift"].copy_((-mean * scale).float())
            self.run_layer(i, stream)

    def launches_per_forward(self):
        # per layer: BinActiv (one or two kernels), conv; plus one kernel per projection shortcut
        act = sum(B.xnor_binactiv_launches(L["desc"], True) for L in self.layers)
        return act + len(self.layers) + len(self.proj)

    def macs(self):
        return sum(wl.macs(s) for s in self.shapes)
