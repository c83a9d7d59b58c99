// k-bit BinActiv: launcher-side queries (internal).
#pragma once
#include "common.cuh"

namespace xnor {

// Kernels launch_binactiv_kbit launches for this shape (1 or 2).
int binactiv_kbit_launch_count(const ConvGeom &g, bool has_bn, int kbits);

}  // namespace xnor
