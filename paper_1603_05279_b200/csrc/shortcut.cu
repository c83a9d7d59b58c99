// Full-precision 1x1 strided convolution without bias (ResNet projection
// shortcut, Section 4.2): out[n][co][oy][ox] = sum_c x[n][c][oy*s][ox*s] w[co][c].
#include "common.cuh"

namespace xnor {

namespace {

constexpr int SP = 64;   // output pixels per block (flat within one image)
constexpr int SF = 64;   // filters per block
constexpr int SK = 16;   // channels per shared-memory step

__global__ void __launch_bounds__(256)
shortcut_conv1x1_kernel(const float *__restrict__ x, const float *__restrict__ w, int C, int H,
                        int W, int Co, int stride, int Ho, int Wo, int tiles_per_image,
                        float *__restrict__ out) {
  __shared__ float xs[SK][SP];
  __shared__ float ws[SK][SF + 1];
  const int n = blockIdx.x / tiles_per_image;
  const int op0 = (blockIdx.x - n * tiles_per_image) * SP;
  const int co0 = blockIdx.y * SF;
  const int HoWo = Ho * Wo;
  const int tx = threadIdx.x % 16;  // pixel quad
  const int ty = threadIdx.x / 16;  // filter quad
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

  for (int c0 = 0; c0 < C; c0 += SK) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < SK * SP; idx += 256) {
      const int kk = idx / SP, pp = idx - kk * SP;
      const int op = op0 + pp, c = c0 + kk;
      float v = 0.0f;
      if (op < HoWo && c < C) {
        const int oy = op / Wo, ox = op - oy * Wo;
        v = __ldg(x + (((size_t)n * C + c) * H + (size_t)oy * stride) * W + (size_t)ox * stride);
      }
      xs[kk][pp] = v;
    }
    for (int idx = threadIdx.x; idx < SK * SF; idx += 256) {
      const int f = idx / SK, kk = idx - f * SK;
      const int co = co0 + f, c = c0 + kk;
      ws[kk][f] = (co < Co && c < C) ? __ldg(w + (size_t)co * C + c) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SK; ++kk) {
      float xv[4], wv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) xv[i] = xs[kk][tx + 16 * i];
#pragma unroll
      for (int j = 0; j < 4; ++j) wv[j] = ws[kk][ty * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = __fmaf_rn(xv[i], wv[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int co = co0 + ty * 4 + j;
    if (co >= Co) continue;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int op = op0 + tx + 16 * i;
      if (op < HoWo) out[((size_t)n * Co + co) * HoWo + op] = acc[i][j];
    }
  }
}

}  // namespace

cudaError_t launch_shortcut_conv1x1(const float *x, const float *w, int N, int C, int H, int W,
                                    int Co, int stride, float *out, cudaStream_t st) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  const int tiles = (Ho * Wo + SP - 1) / SP;
  const dim3 grid((unsigned)(N * tiles), (unsigned)((Co + SF - 1) / SF));
  shortcut_conv1x1_kernel<<<grid, 256, 0, st>>>(x, w, C, H, W, Co, stride, Ho, Wo, tiles, out);
  return cudaGetLastError();
}

}  // namespace xnor
