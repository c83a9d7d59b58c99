// Backward convolution with a binarised gradient (Section 3.2, "Binary Gradient"): the
// gradient at a convolution's output enters the backward convolution as sign(g) scaled by
// max|g| (of the image), the filters as alpha * sign(W) (Algorithm 1).  The contraction runs
// over the filters co with alpha[co] inside the sum, so it is a convolution of the real-valued
// tensor u = gmax * alpha[co] * sign(g) with +-1 filters: the Binary-Weight form (Eq. 1), run
// on that kernel with the filters transposed and turned by 180 degrees.  This file has the two
// small kernels around it: the per-image maximum and the transposed sign packing.
#include <algorithm>

#include "bgrad.cuh"

namespace xnor {

namespace {

// Non-negative floats order like their bit patterns, so the maximum over blocks is an
// integer atomicMax: exact and independent of the order of arrival.  NaN is skipped.
__global__ void __launch_bounds__(256)
grad_max_kernel(const float *__restrict__ g, size_t per_image, int vec4, float *__restrict__ gmax) {
  const float *gi = g + (size_t)blockIdx.y * per_image;
  float m = 0.0f;
  if (vec4) {
    const float4 *g4 = reinterpret_cast<const float4 *>(gi);
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < per_image / 4; i += (size_t)gridDim.x * 256) {
      const float4 v = __ldg(g4 + i);
      m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
  } else {
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < per_image; i += (size_t)gridDim.x * 256)
      m = fmaxf(m, fabsf(__ldg(gi + i)));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float red[8];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]);
    atomicMax(reinterpret_cast<unsigned int *>(gmax) + blockIdx.y, __float_as_uint(m));
  }
}

// One warp per packed word: lane = channel co of the word, the word is a ballot.
__global__ void __launch_bounds__(256)
binarize_weights_transposed_kernel(const float *__restrict__ w, int Co, int C, int kh, int kw,
                                   int CwT, uint32_t *__restrict__ wT_packed) {
  const int lane = threadIdx.x & 31;
  const int taps = kh * kw, nwords = taps * CwT, npad = (nwords + 1) & ~1;
  const long long total = (long long)C * npad;
  for (long long id = (long long)blockIdx.x * 8 + (threadIdx.x >> 5); id < total; id += (long long)gridDim.x * 8) {
    const int ci = (int)(id / npad), f = (int)(id - (long long)ci * npad);
    uint32_t word = 0u;
    if (f < nwords) {
      const int tap = f / CwT, cw = f - tap * CwT;
      const int ky = tap / kw, kx = tap - ky * kw;
      const int co = cw * 32 + lane;
      const bool in = co < Co;
      const float v = in ? __ldg(w + (((size_t)co * C + ci) * kh + (kh - 1 - ky)) * kw + (kw - 1 - kx)) : -1.0f;
      word = __ballot_sync(0xffffffffu, in && v >= 0.0f);
    }
    if (lane == 0) wT_packed[packed_weight_index(C, ci, f)] = word;
  }
}

}  // namespace

cudaError_t launch_grad_max(const float *g, int N, size_t per_image, float *gmax, cudaStream_t st) {
  if (N > 65535) return cudaErrorInvalidValue;
  cudaError_t e = cudaMemsetAsync(gmax, 0, sizeof(float) * (size_t)N, st);
  if (e != cudaSuccess) return e;
  // enough blocks to fill the GPU whatever the batch, at most one per 4096 values
  const int sms = sm_count_of_current_device();
  const size_t want = (size_t)(8 * sms + N - 1) / (size_t)N;
  const size_t cap = (per_image + 4095) / 4096;
  const unsigned bx = (unsigned)std::max<size_t>(1, std::min(want, cap));
  const int vec4 = (per_image % 4 == 0) ? 1 : 0;     // then every image starts on a 16-byte boundary
  grad_max_kernel<<<dim3(bx, (unsigned)N), 256, 0, st>>>(g, per_image, vec4, gmax);
  return cudaGetLastError();
}

cudaError_t launch_binarize_weights_transposed(const float *w, int Co, int C, int kh, int kw,
                                               uint32_t *wT_packed, cudaStream_t st) {
  const int CwT = (Co + 31) / 32;
  const long long total = (long long)C * ((kh * kw * CwT + 1) & ~1);
  const unsigned grid = (unsigned)std::min<long long>((total + 7) / 8, 4096);
  binarize_weights_transposed_kernel<<<grid, 256, 0, st>>>(w, Co, C, kh, kw, CwT, wT_packed);
  return cudaGetLastError();
}

}  // namespace xnor
