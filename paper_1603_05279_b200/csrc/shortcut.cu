// Full-precision 1x1 strided convolution without bias (ResNet projection
// shortcut, Section 4.2): out[n][co][oy][ox] = sum_c x[n][c][oy*s][ox*s] w[co][c].
#include "common.cuh"

namespace xnor {

namespace {

constexpr int SP = 128;  // output pixels per block (flat over images and pixels)
constexpr int SF = 64;   // filters per block
constexpr int SK = 32;   // channels per shared-memory step

// 256 threads; thread (tx, ty) owns pixels 4 tx .. 4 tx + 3 and 64 + 4 tx .. 64 + 4 tx + 3 and
// filters 4 ty .. 4 ty + 3: each step of the inner loop is three 16-byte shared-memory reads
// (conflict-free: a quarter warp reads 128 contiguous bytes) for 32 multiply-adds.  The next
// step's operands travel global -> registers while the current step is computed.
__global__ void __launch_bounds__(256)
shortcut_conv1x1_kernel(const float *__restrict__ x, const float *__restrict__ w, int C, int H,
                        int W, int Co, int stride, int Ho, int Wo, long long total_pix,
                        float *__restrict__ out) {
  __shared__ __align__(16) float xs[2][SK][SP];
  __shared__ __align__(16) float ws[2][SK][SF];
  const long long op0 = (long long)blockIdx.x * SP;
  const int co0 = blockIdx.y * SF;
  const int HoWo = Ho * Wo;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

  // staging duties.  x: one pixel, 16 channels (lk, lk + 2, ...); w: one filter, 8 consecutive
  // channels (two 16-byte loads when C % 4 == 0)
  const int lp = threadIdx.x & 127, lk = threadIdx.x >> 7;
  const long long lgp = op0 + lp;
  const bool lp_on = lgp < total_pix;
  const long long ln = lp_on ? lgp / HoWo : 0;
  const int lop = lp_on ? (int)(lgp - ln * HoWo) : 0;
  const int loy = lop / Wo, lox = lop - loy * Wo;
  const float *xsrc = x + ((size_t)ln * C * H + (size_t)loy * stride) * W + (size_t)lox * stride;
  const size_t plane = (size_t)H * W;
  const int lf = threadIdx.x >> 2, lc = (threadIdx.x & 3) * 8;
  const bool lf_on = co0 + lf < Co;
  const float *wsrc = w + (size_t)(lf_on ? co0 + lf : 0) * C;
  const bool wvec = (C & 3) == 0;
  float xr[16], wr[8];
  auto fetch = [&](int c0) {
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const int cx = c0 + lk + 2 * q;
      xr[q] = (lp_on && cx < C) ? __ldg(xsrc + (size_t)cx * plane) : 0.0f;
    }
    if (wvec && lf_on && c0 + lc + 8 <= C) {
      const float4 a = __ldg(reinterpret_cast<const float4 *>(wsrc + c0 + lc));
      const float4 b = __ldg(reinterpret_cast<const float4 *>(wsrc + c0 + lc + 4));
      wr[0] = a.x; wr[1] = a.y; wr[2] = a.z; wr[3] = a.w;
      wr[4] = b.x; wr[5] = b.y; wr[6] = b.z; wr[7] = b.w;
    } else {
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int cw = c0 + lc + q;
        wr[q] = (lf_on && cw < C) ? __ldg(wsrc + cw) : 0.0f;
      }
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int q = 0; q < 16; ++q) xs[buf][lk + 2 * q][lp] = xr[q];
#pragma unroll
    for (int q = 0; q < 8; ++q) ws[buf][lc + q][lf] = wr[q];
  };
  fetch(0);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int c0 = 0; c0 < C; c0 += SK) {
    if (c0 + SK < C) fetch(c0 + SK);          // next step's values are in flight during the math
#pragma unroll 8
    for (int kk = 0; kk < SK; ++kk) {
      const float4 x0 = *reinterpret_cast<const float4 *>(&xs[buf][kk][tx * 4]);
      const float4 x1 = *reinterpret_cast<const float4 *>(&xs[buf][kk][64 + tx * 4]);
      const float4 wv = *reinterpret_cast<const float4 *>(&ws[buf][kk][ty * 4]);
      const float xa[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
      const float wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = __fmaf_rn(xa[i], wa[j], acc[i][j]);
    }
    if (c0 + SK < C) {
      stash(buf ^ 1);
      __syncthreads();
      buf ^= 1;
    }
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    // four consecutive pixels of the flat index: one image and 16-byte aligned when H_out*W_out
    // is a multiple of 4, else each pixel finds its own image
    const long long gp = op0 + 64 * h + tx * 4;
    if (gp >= total_pix) continue;
    const bool vec = (HoWo & 3) == 0;
    const long long n0 = gp / HoWo;
    const int p0 = (int)(gp - n0 * HoWo);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int co = co0 + ty * 4 + j;
      if (co >= Co) continue;
      if (vec) {
        float *dst = out + ((size_t)n0 * Co + co) * HoWo + p0;
        *reinterpret_cast<float4 *>(dst) = make_float4(acc[4 * h][j], acc[4 * h + 1][j],
                                                       acc[4 * h + 2][j], acc[4 * h + 3][j]);
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (gp + i < total_pix) {
            const long long ni = p0 + i < HoWo ? n0 : (gp + i) / HoWo;
            const int pi = (int)(gp + i - ni * HoWo);
            out[((size_t)ni * Co + co) * HoWo + pi] = acc[4 * h + i][j];
          }
        }
      }
    }
  }
}

}  // namespace

cudaError_t launch_shortcut_conv1x1(const float *x, const float *w, int N, int C, int H, int W,
                                    int Co, int stride, float *out, cudaStream_t st) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  const long long total_pix = (long long)N * Ho * Wo;
  const long long tiles = (total_pix + SP - 1) / SP;
  if (tiles > 0x7FFFFFFFll) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)tiles, (unsigned)((Co + SF - 1) / SF));
  shortcut_conv1x1_kernel<<<grid, 256, 0, st>>>(x, w, C, H, W, Co, stride, Ho, Wo, total_pix, out);
  return cudaGetLastError();
}

}  // namespace xnor
