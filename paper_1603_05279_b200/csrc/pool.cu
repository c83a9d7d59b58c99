// The Pool layer that closes the block (Section 3.2, "Training XNOR-Networks": BatchNorm,
// BinActiv, BinConv, Pool, with an optional ReLU after the binary convolution): max pooling
// of BinConv's fp32 output.  Taps outside the image take no part in the maximum.
#include <algorithm>

#include "common.cuh"

namespace xnor {

namespace {

constexpr int kPoolThreads = 256;

// Exact n / d for n < 2^31: q = (n * m) >> (31 + s) with m = ceil(2^(31+s) / d), s = ceil(log2 d).
struct Magic { uint32_t m; int s; };
__device__ __forceinline__ uint32_t fast_div(uint32_t n, Magic g) {
  return (uint32_t)(((uint64_t)n * g.m) >> (31 + g.s));
}

// A thread per output (consecutive threads = consecutive outputs of a plane, so stores are
// coalesced); its window comes through the read-only cache, where the overlapping windows of
// neighbouring outputs meet, so HBM sees each input element once.  (A variant that staged
// whole planes in shared memory first was measured slower: 1.9 against 2.3-2.5 TB/s.)
template <bool kRelu>
__global__ void __launch_bounds__(kPoolThreads)
maxpool_kernel(const float *__restrict__ x, long long total_out, int H, int W, int k, int stride,
               int pad, int Ho, int Wo, Magic div_howo, Magic div_wo, float *__restrict__ out) {
  const int HoWo = Ho * Wo;
  // chunks of 2^30 outputs keep the index arithmetic in 32 bits
  for (long long base = 0; base < total_out; base += (1ll << 30)) {
    const uint32_t count = (uint32_t)min(total_out - base, 1ll << 30);
    const long long plane0 = base / HoWo;               // base is not a multiple of HoWo in general:
    const uint32_t off0 = (uint32_t)(base - plane0 * HoWo);   // outputs of the chunk start off0 into plane0
    for (uint32_t i = blockIdx.x * kPoolThreads + threadIdx.x; i < count;
         i += gridDim.x * kPoolThreads) {
      const uint32_t o = i + off0;                       // < 2^31
      const uint32_t pl = fast_div(o, div_howo);
      const int r = (int)(o - pl * (uint32_t)HoWo);
      const int oy = (int)fast_div((uint32_t)r, div_wo), ox = r - oy * Wo;
      const int y0 = max(oy * stride - pad, 0), y1 = min(oy * stride - pad + k, H);
      const int x0 = max(ox * stride - pad, 0), x1 = min(ox * stride - pad + k, W);
      const float *t = x + (size_t)(plane0 + pl) * H * W;
      float m = __ldg(t + (size_t)y0 * W + x0);
      for (int iy = y0; iy < y1; ++iy)
        for (int ix = x0; ix < x1; ++ix) m = fmaxf(m, __ldg(t + (size_t)iy * W + ix));
      out[base + i] = kRelu ? fmaxf(m, 0.0f) : m;
    }
  }
}

}  // namespace

cudaError_t launch_maxpool2d(const float *x, int N, int C, int H, int W, int k, int stride, int pad,
                             bool relu, float *out, cudaStream_t st) {
  const int Ho = (H + 2 * pad - k) / stride + 1, Wo = (W + 2 * pad - k) / stride + 1;
  if ((long long)Ho * Wo >= (1ll << 30)) return cudaErrorInvalidValue;
  const long long total = (long long)N * C * Ho * Wo;
  const int sms = sm_count_of_current_device();
  auto magic = [](uint32_t d) {
    Magic g;
    g.s = 0;
    while ((1u << g.s) < d) ++g.s;
    g.m = (uint32_t)((((unsigned long long)1 << (31 + g.s)) + d - 1) / d);
    return g;
  };
  const Magic dh = magic((uint32_t)(Ho * Wo)), dw = magic((uint32_t)Wo);
  const unsigned grid = (unsigned)std::min<long long>((total + kPoolThreads - 1) / kPoolThreads,
                                                      16ll * sms);
  if (relu)
    maxpool_kernel<true><<<grid, kPoolThreads, 0, st>>>(x, total, H, W, k, stride, pad, Ho, Wo, dh, dw, out);
  else
    maxpool_kernel<false><<<grid, kPoolThreads, 0, st>>>(x, total, H, W, k, stride, pad, Ho, Wo, dh, dw, out);
  return cudaGetLastError();
}

}  // namespace xnor
