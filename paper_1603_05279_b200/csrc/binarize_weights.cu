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
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float *wf = w + (size_t)co * n;
  // A warp builds one packed word at a time: lane = channel within the word, the word is a
  // ballot of (w >= 0).  No atomics, no divisions per weight.
  double l1 = 0.0;
  int tap = 0, cw = warp;                      // word f = tap * Cw + cw, visited in steps of 8
  while (cw >= Cw) { cw -= Cw; ++tap; }
  for (int f = warp; f < nwords; f += kThreads / 32) {
    const int ci = cw * 32 + lane;
    const bool in = ci < C;
    const float v = in ? __ldg(wf + (size_t)ci * taps + tap) : -1.0f;
    if (in) l1 += fabs((double)v);
    const uint32_t word = __ballot_sync(0xffffffffu, in && v >= 0.0f);
    if (lane == 0) words[f] = word;
    cw += kThreads / 32;
    while (cw >= Cw) { cw -= Cw; ++tap; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
  if (lane == 0) red[warp] = l1;
  __syncthreads();
  if (threadIdx.x == 0) {
    double sum = 0.0;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) sum += red[i];
    alpha[co] = (float)(sum / (double)n);
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
