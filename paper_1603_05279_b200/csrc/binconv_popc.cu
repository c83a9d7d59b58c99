// BinConv on CUDA cores (Eq. 11): for every output pixel and filter,
//   acc = sum over in-image taps of (C_in - 2 popcount(a xor b)),
// then out = acc * K * alpha (+ residual).  Works for every supported shape.
#include "common.cuh"

namespace xnor {

namespace {

constexpr int TP = 64;    // output pixels per block, flat (oy*Wo + ox) within one image
constexpr int TF = 64;    // filters per block
constexpr int FPT = 16;   // filters per thread
constexpr int kThreads = TP * (TF / FPT);

struct PopcParams {
  int C, H, W, Co, kh, kw, stride, pad, Ho, Wo, Cw;
  int tiles_per_image;  // ceil(Ho*Wo / TP)
  int PW;               // patch width  = (Wo-1)*stride + kw   (input columns -pad .. )
  int PHmax;            // patch rows staged per block
  int PP;               // PHmax * PW
  int cwc;              // channel words per shared-memory chunk
};

__global__ void __launch_bounds__(kThreads)
binconv_popc_kernel(const uint32_t *__restrict__ xp, const uint32_t *__restrict__ wp,
                    const float *__restrict__ alpha, const float *__restrict__ K,
                    const float *residual, PopcParams P, EpiOpts epi, float *out, int32_t *acc_out) {
  extern __shared__ uint32_t smem[];
  const int taps = P.kh * P.kw;
  uint32_t *patch = smem;                       // [cwc][PP]
  uint32_t *wts = smem + (size_t)P.cwc * P.PP;  // [TF][taps][cwc]

  const int n = blockIdx.x / P.tiles_per_image;
  const int tile = blockIdx.x - n * P.tiles_per_image;
  const int co0 = blockIdx.y * TF;
  const int HoWo = P.Ho * P.Wo;
  const int op0 = tile * TP;
  const int op_last = min(op0 + TP, HoWo) - 1;
  const int oy_first = op0 / P.Wo;
  const int oy_last = op_last / P.Wo;
  const int iy0 = oy_first * P.stride - P.pad;             // input row of patch row 0
  const int PH = (oy_last - oy_first) * P.stride + P.kh;   // rows actually needed (<= PHmax)

  const int pl = threadIdx.x % TP;   // pixel lane
  const int fg = threadIdx.x / TP;   // filter group (warp-uniform)
  const int op = op0 + pl;
  const bool live = op < HoWo;
  const int oy = live ? op / P.Wo : oy_first;
  const int ox = live ? op - oy * P.Wo : 0;
  const int pr0 = (oy - oy_first) * P.stride;  // patch row of tap ky = 0
  const int pc0 = ox * P.stride;               // patch column of tap kx = 0

  int pops[FPT];
#pragma unroll
  for (int f = 0; f < FPT; ++f) pops[f] = 0;
  int nvalid = 0;

  for (int cw0 = 0; cw0 < P.Cw; cw0 += P.cwc) {
    const int cwn = min(P.cwc, P.Cw - cw0);
    __syncthreads();
    // stage the input patch, zero outside the image
    for (int idx = threadIdx.x; idx < PH * P.PW * cwn; idx += kThreads) {
      const int cw = idx % cwn;
      const int pix = idx / cwn;
      const int r = pix / P.PW, cx = pix - r * P.PW;
      const int iy = iy0 + r, ix = cx - P.pad;
      uint32_t v = 0u;
      if (iy >= 0 && iy < P.H && ix >= 0 && ix < P.W)
        v = __ldg(xp + (((size_t)n * P.H + iy) * P.W + ix) * P.Cw + cw0 + cw);
      patch[cw * P.PP + pix] = v;
    }
    // stage the filter tile
    for (int idx = threadIdx.x; idx < TF * taps * cwn; idx += kThreads) {
      const int cw = idx % cwn;
      const int ft = idx / cwn;           // f*taps + tap
      const int f = ft / taps;
      uint32_t v = 0u;
      if (co0 + f < P.Co)
        v = __ldg(wp + packed_weight_index(P.Co, co0 + f, (ft - f * taps) * P.Cw + cw0 + cw));
      wts[ft * P.cwc + cw] = v;
    }
    __syncthreads();
    if (live) {
      for (int ky = 0; ky < P.kh; ++ky) {
        const int iy = oy * P.stride + ky - P.pad;
        if (iy < 0 || iy >= P.H) continue;
        for (int kx = 0; kx < P.kw; ++kx) {
          const int ix = ox * P.stride + kx - P.pad;
          if (ix < 0 || ix >= P.W) continue;      // padded tap: contributes 0
          if (cw0 == 0) ++nvalid;
          const int pidx = (pr0 + ky) * P.PW + pc0 + kx;
          const uint32_t *wt = wts + ((size_t)(fg * FPT) * taps + ky * P.kw + kx) * P.cwc;
          for (int cw = 0; cw < cwn; ++cw) {
            const uint32_t a = patch[cw * P.PP + pidx];
#pragma unroll
            for (int f = 0; f < FPT; ++f)
              pops[f] += __popc(a ^ wt[(size_t)f * taps * P.cwc + cw]);
          }
        }
      }
    }
  }
  if (!live) return;
  const float kv = __ldg(K + (size_t)n * HoWo + op);
#pragma unroll
  for (int f = 0; f < FPT; ++f) {
    const int co = co0 + fg * FPT + f;
    if (co >= P.Co) break;
    const int acc = nvalid * P.C - 2 * pops[f];
    const size_t o = ((size_t)n * P.Co + co) * HoWo + op;
    float v = __fmul_rn(__fmul_rn((float)acc, kv), __fmul_rn(__ldg(alpha + co), epi.out_scale));
    if (residual) v += residual[o];
    if (epi.relu) v = fmaxf(v, 0.0f);
    out[o] = v;
    if (acc_out) acc_out[o] = (epi.acc_accum ? acc_out[o] : 0) + (acc << epi.acc_shift);
  }
}

}  // namespace

// Shapes the CUDA-core engine covers: one channel word of the input patch and of the filter
// tile must fit its 96 KB of shared memory.
bool binconv_popc_supported(const ConvGeom &g) {
  const long long PW = (long long)(g.Wo - 1) * g.stride + g.kw;
  long long rows = (TP - 1 + g.Wo - 1) / g.Wo + 1;
  if (rows > g.Ho) rows = g.Ho;
  const long long PP = ((rows - 1) * g.stride + g.kh) * PW;
  const long long words_per_cw = PP + (long long)TF * g.kh * g.kw;
  return words_per_cw <= (long long)(96 * 1024 / sizeof(uint32_t)) &&
         (long long)g.N * ((g.Ho * g.Wo + TP - 1) / TP) < (1ll << 31) && (g.Co + TF - 1) / TF <= 65535;
}

cudaError_t launch_binconv_popc(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                                const float *K, const float *residual, const ConvGeom &g,
                                const EpiOpts &epi, float *out, int32_t *acc_out, cudaStream_t st) {
  PopcParams P;
  P.C = g.C; P.H = g.H; P.W = g.W; P.Co = g.Co; P.kh = g.kh; P.kw = g.kw;
  P.stride = g.stride; P.pad = g.pad; P.Ho = g.Ho; P.Wo = g.Wo; P.Cw = g.Cw;
  const int HoWo = g.Ho * g.Wo;
  P.tiles_per_image = (HoWo + TP - 1) / TP;
  P.PW = (g.Wo - 1) * g.stride + g.kw;
  int rows = (TP - 1 + g.Wo - 1) / g.Wo + 1;   // output rows a run of TP flat pixels can touch
  if (rows > g.Ho) rows = g.Ho;
  P.PHmax = (rows - 1) * g.stride + g.kh;
  P.PP = P.PHmax * P.PW;
  const int taps = g.kh * g.kw;
  const size_t words_per_cw = (size_t)P.PP + (size_t)TF * taps;
  const size_t budget = 96 * 1024 / sizeof(uint32_t);
  int cwc = (int)(budget / words_per_cw);
  if (cwc < 1) return cudaErrorInvalidValue;
  if (cwc > g.Cw) cwc = g.Cw;
  if (cwc > 8) cwc = 8;
  P.cwc = cwc;
  const size_t smem = words_per_cw * cwc * sizeof(uint32_t);
  static bool attr_flags[64] = {};
  bool &attr_set = attr_done_for_current_device(attr_flags);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(binconv_popc_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  const dim3 grid((unsigned)(g.N * P.tiles_per_image), (unsigned)((g.Co + TF - 1) / TF));
  binconv_popc_kernel<<<grid, kThreads, smem, st>>>(xp, wp, alpha, K, residual, P, epi, out, acc_out);
  return cudaGetLastError();
}

}  // namespace xnor
