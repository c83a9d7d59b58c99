// Weight binarisation: B = sign(W) bit-packed along channels (word-pair-major), alpha = ||W||_1/n
// per filter (Section 3.1, Eq. 4 and Eq. 6).  One thread block per filter.
#include "common.cuh"

namespace xnor {

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
binarize_weights_kernel(const float *__restrict__ w, int Co, int C, int taps, int Cw,
                        uint32_t *__restrict__ w_packed, float *__restrict__ alpha) {
  extern __shared__ uint32_t words[];  // [taps][Cw]
  __shared__ double red[kThreads / 32];
  const int co = blockIdx.x;
  const int n = C * taps;
  const int nwords = taps * Cw;
  for (int j = threadIdx.x; j < nwords; j += kThreads) words[j] = 0u;
  __syncthreads();

  const float *wf = w + (size_t)co * n;
  double l1 = 0.0;
  for (int i = threadIdx.x; i < n; i += kThreads) {   // i = ci*taps + tap
    const float v = wf[i];
    l1 += fabs((double)v);
    if (v >= 0.0f) {
      const int ci = i / taps, tap = i - ci * taps;
      atomicOr(&words[tap * Cw + (ci >> 5)], 1u << (ci & 31));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = l1;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) s += red[i];
    alpha[co] = (float)(s / (double)n);
  }
  // word-pair-major layout (see packed_weight_index); an odd word count is padded with 0
  for (int j = threadIdx.x; j < ((nwords + 1) & ~1); j += kThreads)
    w_packed[packed_weight_index(Co, co, j)] = j < nwords ? words[j] : 0u;
}

}  // namespace

cudaError_t launch_binarize_weights(const float *w, int Co, int C, int kh, int kw,
                                    uint32_t *w_packed, float *alpha, cudaStream_t st) {
  const int taps = kh * kw, Cw = (C + 31) / 32;
  const size_t smem = (size_t)taps * Cw * sizeof(uint32_t);
  if (smem > 48 * 1024) return cudaErrorInvalidValue;
  binarize_weights_kernel<<<Co, kThreads, smem, st>>>(w, Co, C, taps, Cw, w_packed, alpha);
  return cudaGetLastError();
}

}  // namespace xnor
