// Full-precision 1x1 strided convolution without bias (ResNet projection
// shortcut, Section 4.2): out[n][co][oy][ox] = sum_c x[n][c][oy*s][ox*s] w[co][c].
#include "common.cuh"

namespace xnor {

namespace {

constexpr int SP = 64;   // output pixels per block (flat within one image)
constexpr int SF = 64;   // filters per block
constexpr int SK = 16;   // channels per shared-memory step

// 256 threads; thread (tx, ty) owns pixels 4 tx .. 4 tx + 3 and filters 4 ty .. 4 ty + 3, so
// each step of the inner loop is two 16-byte shared-memory reads for 16 multiply-adds.
__global__ void __launch_bounds__(256)
shortcut_conv1x1_kernel(const float *__restrict__ x, const float *__restrict__ w, int C, int H,
                        int W, int Co, int stride, int Ho, int Wo, int tiles_per_image,
                        float *__restrict__ out) {
  __shared__ __align__(16) float xs[2][SK][SP];
  __shared__ __align__(16) float ws[2][SK][SF];
  const int n = blockIdx.x / tiles_per_image;
  const int op0 = (blockIdx.x - n * tiles_per_image) * SP;
  const int co0 = blockIdx.y * SF;
  const int HoWo = Ho * Wo;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

  // this thread's staging duties: 4 x values (one pixel, 4 channels apart) and 4 w values
  const int lp = threadIdx.x & 63, lk = threadIdx.x >> 6;          // pixel, channel 0..3 (+4, +8, +12)
  const int lop = op0 + lp;
  const bool lp_on = lop < HoWo;
  const int loy = lp_on ? lop / Wo : 0, lox = lp_on ? lop - loy * Wo : 0;
  const float *xsrc = x + ((size_t)n * C * H + (size_t)loy * stride) * W + (size_t)lox * stride;
  const int lf = threadIdx.x >> 2, lc = threadIdx.x & 3;            // filter, channel 0..3 (+4, ...)
  const bool lf_on = co0 + lf < Co;
  const float *wsrc = w + (size_t)(lf_on ? co0 + lf : 0) * C;
  float xr[4], wr[4];
  auto fetch = [&](int c0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int cx = c0 + lk + 4 * q, cw = c0 + lc + 4 * q;
      xr[q] = (lp_on && cx < C) ? __ldg(xsrc + (size_t)cx * H * W) : 0.0f;
      wr[q] = (lf_on && cw < C) ? __ldg(wsrc + cw) : 0.0f;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      xs[buf][lk + 4 * q][lp] = xr[q];
      ws[buf][lc + 4 * q][lf] = wr[q];
    }
  };
  fetch(0);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int c0 = 0; c0 < C; c0 += SK) {
    if (c0 + SK < C) fetch(c0 + SK);          // next step's values are in flight during the math
#pragma unroll
    for (int kk = 0; kk < SK; ++kk) {
      const float4 xv = *reinterpret_cast<const float4 *>(&xs[buf][kk][tx * 4]);
      const float4 wv = *reinterpret_cast<const float4 *>(&ws[buf][kk][ty * 4]);
      const float xa[4] = {xv.x, xv.y, xv.z, xv.w}, wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = __fmaf_rn(xa[i], wa[j], acc[i][j]);
    }
    if (c0 + SK < C) {
      stash(buf ^ 1);
      __syncthreads();
      buf ^= 1;
    }
  }
  const int op = op0 + tx * 4;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int co = co0 + ty * 4 + j;
    if (co >= Co) continue;
    float *dst = out + ((size_t)n * Co + co) * HoWo + op;
    if (op + 3 < HoWo && (HoWo & 3) == 0) {
      *reinterpret_cast<float4 *>(dst) = make_float4(acc[0][j], acc[1][j], acc[2][j], acc[3][j]);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (op + i < HoWo) dst[i] = acc[i][j];
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
