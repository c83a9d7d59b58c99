"""CPU oracle of the XNOR-Net forward block (test infrastructure only).

Thin numpy/ctypes binding over ``xnor_oracle.c``; all arithmetic lives in the
C file.  Nothing in the CUDA package imports this module, and this module
imports nothing from it.
"""
from .binding import (  # noqa: F401
    build,
    lib_path,
    num_threads,
    set_num_threads,
    bn_affine,
    sign,
    channel_abs_mean,
    box_filter,
    binarize_weights,
    binconv_acc,
    scale_output,
    xnor_block,
    xnor_block_ex,
    box_filter_valid_taps,
    relu,
    quantize_k,
    scale_output_k,
    round_bf16,
    bwn_conv,
    binary_gradient_backward,
    shortcut_conv1x1,
    maxpool2d,
    speedup_model,
    out_extent,
)
