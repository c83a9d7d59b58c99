// Launchers of the backward convolution with a binarised gradient (internal).
#pragma once
#include "common.cuh"

namespace xnor {

// gmax[n] = max |g| over image n's `per_image` values (gmax is cleared first).
cudaError_t launch_grad_max(const float *g, int N, size_t per_image, float *gmax, cudaStream_t st);

// Sign bits of the filters as the backward convolution contracts them: filter ci of the result
// has the channels co and the taps turned by 180 degrees,
// bit(ci; co, ky, kx) = (w[co][ci][kh-1-ky][kw-1-kx] >= 0); word-pair-major like w_packed.
cudaError_t launch_binarize_weights_transposed(const float *w, int Co, int C, int kh, int kw,
                                               uint32_t *wT_packed, cudaStream_t st);

// The pixel stream of the Binary-Weight convolution (geometry gb: the backward convolution's)
// filled with sign(g) * bf16(gmax[n] * alpha[co]).
cudaError_t launch_bwn_prepare_grad(const float *g, const float *alpha, const float *gmax,
                                    const ConvGeom &gb, uint16_t *g_stream, cudaStream_t st);

}  // namespace xnor
