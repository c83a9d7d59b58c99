// BatchNorm affine + BinActiv (Section 3.2): sign bits packed along channels,
// A = channel mean of |y|, then K = box filter of zero-padded A at the
// convolution's output positions.
#include "common.cuh"

namespace xnor {

namespace {

constexpr int kPix = 32;      // pixels per block (one warp wide)
constexpr int kMaxGroups = 8; // warps per block; each owns a subset of the channel words

// Block = kPix consecutive pixels (flat over n,h,w) x G warps.  Lane = pixel, so
// each warp-level load of one channel is a contiguous 128-byte run of x.  Warp
// g packs channel words g, g+G, ...  Words are staged in shared memory and
// written as one contiguous run of kPix*Cw words.
template <bool kHasBN>
__global__ void __launch_bounds__(kPix * kMaxGroups)
binactiv_pack_kernel(const float *__restrict__ x, const float *__restrict__ scale,
                     const float *__restrict__ shift, long long total_pix, int C, int HW, int Cw,
                     uint32_t *__restrict__ x_packed, float *__restrict__ A) {
  extern __shared__ uint32_t tile[];            // [kPix][Cw]
  __shared__ float sabs[kMaxGroups][kPix];
  const int lane = threadIdx.x, g = threadIdx.y, G = blockDim.y;
  const long long gp0 = (long long)blockIdx.x * kPix;
  const long long gp = gp0 + lane;
  const bool live = gp < total_pix;
  const long long n = live ? gp / HW : 0;
  const int p = live ? (int)(gp - n * HW) : 0;
  const float *xb = x + (size_t)n * C * HW + p;

  float asum = 0.0f;
  for (int cw = g; cw < Cw; cw += G) {
    const int c0 = cw * 32;
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const int c = c0 + j;
      v[j] = (live && c < C) ? __ldcs(xb + (size_t)c * HW) : -1.0f;
    }
    uint32_t word = 0u;
    float part = 0.0f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const int c = c0 + j;
      if (c < C) {
        float y = v[j];
        if (kHasBN) y = __fmaf_rn(__ldg(scale + c), y, __ldg(shift + c));
        word |= (y >= 0.0f ? 1u : 0u) << j;
        part += fabsf(y);
      }
    }
    asum += part;
    tile[lane * Cw + cw] = word;
  }
  sabs[g][lane] = asum;
  __syncthreads();
  if (g == 0 && live) {
    float s = 0.0f;
    for (int i = 0; i < G; ++i) s += sabs[i][lane];
    A[gp] = s / (float)C;
  }
  const long long nw = (total_pix - gp0 < kPix ? total_pix - gp0 : kPix) * Cw;
  uint32_t *dst = x_packed + (size_t)gp0 * Cw;
  for (int j = g * kPix + lane; j < nw; j += G * kPix) dst[j] = tile[j];
}

__global__ void box_filter_kernel(const float *__restrict__ A, int N, int H, int W, int kh,
                                  int kw, int stride, int pad, int Ho, int Wo,
                                  float *__restrict__ K) {
  const long long total = (long long)N * Ho * Wo;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int ox = (int)(i % Wo);
  const int oy = (int)((i / Wo) % Ho);
  const long long n = i / ((long long)Wo * Ho);
  const float *a = A + (size_t)n * H * W;
  float s = 0.0f;
  for (int ky = 0; ky < kh; ++ky) {
    const int iy = oy * stride + ky - pad;
    if (iy < 0 || iy >= H) continue;
    for (int kx = 0; kx < kw; ++kx) {
      const int ix = ox * stride + kx - pad;
      if (ix < 0 || ix >= W) continue;
      s += __ldg(a + iy * W + ix);
    }
  }
  K[i] = s / (float)(kh * kw);
}

}  // namespace

cudaError_t launch_binactiv(const float *x, const float *scale, const float *shift,
                            const ConvGeom &g, uint32_t *x_packed, float *A, float *K,
                            cudaStream_t st) {
  const long long total_pix = (long long)g.N * g.H * g.W;
  const int G = g.Cw < kMaxGroups ? g.Cw : kMaxGroups;
  const dim3 block(kPix, G);
  const unsigned grid = (unsigned)((total_pix + kPix - 1) / kPix);
  const size_t smem = (size_t)kPix * g.Cw * sizeof(uint32_t);
  if (scale)
    binactiv_pack_kernel<true><<<grid, block, smem, st>>>(x, scale, shift, total_pix, g.C,
                                                          g.H * g.W, g.Cw, x_packed, A);
  else
    binactiv_pack_kernel<false><<<grid, block, smem, st>>>(x, scale, shift, total_pix, g.C,
                                                           g.H * g.W, g.Cw, x_packed, A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const long long total_k = (long long)g.N * g.Ho * g.Wo;
  box_filter_kernel<<<(unsigned)((total_k + 255) / 256), 256, 0, st>>>(
      A, g.N, g.H, g.W, g.kh, g.kw, g.stride, g.pad, g.Ho, g.Wo, K);
  return cudaGetLastError();
}


// ---------------------------------------------------------------------------
// xnor_binactiv_static: the same two kernels, with the A plane kept in a
// fixed array of this library instead of a caller buffer.
namespace {

constexpr size_t kStaticPixels = XNOR_BINACTIV_STATIC_MAX_PIXELS;
constexpr int kMaxDevices = 64;

// Lives in the device memory of every GPU that loads the library, until exit.
static __device__ __align__(256) float g_static_A[kStaticPixels];

// In host code `g_static_A` is only a handle for the runtime; the device
// address has to be asked for, per device, with that device current.
float *g_static_A_ptr[kMaxDevices] = {};

cudaError_t static_A_address(float **ptr) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_static_A_ptr[dev] == nullptr) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_A);
    if (e != cudaSuccess) return e;
    g_static_A_ptr[dev] = static_cast<float *>(p);
  }
  *ptr = g_static_A_ptr[dev];
  return cudaSuccess;
}

}  // namespace

size_t binactiv_static_max_pixels() { return kStaticPixels; }

cudaError_t launch_binactiv_static(const float *x, const float *scale, const float *shift,
                                   const ConvGeom &g, uint32_t *x_packed, float *K,
                                   cudaStream_t st) {
  float *A = nullptr;
  cudaError_t e = static_A_address(&A);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
  // every A value the box filter reads is written by the pack kernel of this call first,
  // so nothing left by an earlier call is ever used and nothing needs clearing
  return launch_binactiv(x, scale, shift, g, x_packed, A, K, st);
}

}  // namespace xnor
