// Shared declarations of the CUDA translation units of libxnor (internal).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "xnor.h"

namespace xnor {

struct ConvGeom {
  int N, C, H, W, Co, kh, kw, stride, pad, Ho, Wo, Cw;
  int flags;      // XNOR_FLAG_* of the descriptor
};

// What the BinConv epilogues do beyond Eq. 11's D K alpha (+ residual).
struct EpiOpts {
  int relu;          // max(v, 0) on the stored value
  float out_scale;   // v = D K (alpha out_scale); 1: as Eq. 11
  int acc_shift;     // acc_out receives D << acc_shift ...
  int acc_accum;     // ... added to what acc_out holds (1) or stored (0)
};
inline EpiOpts default_epi(const ConvGeom &g) {
  EpiOpts e;
  e.relu = (g.flags & XNOR_FLAG_RELU) ? 1 : 0;
  e.out_scale = 1.0f;
  e.acc_shift = 0;
  e.acc_accum = 0;
  return e;
}

inline ConvGeom make_geom(const xnor_conv_desc &d) {
  ConvGeom g;
  g.N = d.N; g.C = d.C_in; g.H = d.H; g.W = d.W; g.Co = d.C_out;
  g.kh = d.k_h; g.kw = d.k_w; g.stride = d.stride; g.pad = d.pad;
  g.Ho = (d.H + 2 * d.pad - d.k_h) / d.stride + 1;
  g.Wo = (d.W + 2 * d.pad - d.k_w) / d.stride + 1;
  g.Cw = (d.C_in + 31) / 32;
  g.flags = d.flags;
  return g;
}

// Packed weights are stored word-pair-major so that the convolution kernels read them
// coalesced: with f = tap * Cw + cw the index of a word inside a filter (tap = ky * k_w + kx),
// word f of filter co is element ((f / 2) * C_out + co) * 2 + f % 2.  Words 2j and 2j+1 of all
// filters (one 64-channel step of the contraction) are contiguous.
__host__ __device__ inline size_t packed_weight_index(int Co, int co, int f) {
  return ((size_t)(f >> 1) * Co + co) * 2 + (f & 1);
}

// Launchers: return the cudaError_t of the launch (cudaGetLastError, cleared).
cudaError_t launch_binarize_weights(const float *w, int Co, int C, int kh, int kw,
                                    uint32_t *w_packed, float *alpha, cudaStream_t st);
cudaError_t launch_binactiv(const float *x, const float *scale, const float *shift,
                            const ConvGeom &g, uint32_t *x_packed, float *A, float *K,
                            cudaStream_t st);
// Same, with A in the library's own fixed array (N*H*W <= binactiv_static_max_pixels()).
size_t binactiv_static_max_pixels();
cudaError_t launch_binactiv_static(const float *x, const float *scale, const float *shift,
                                   const ConvGeom &g, uint32_t *x_packed, float *K,
                                   cudaStream_t st);
bool binactiv_supported(const ConvGeom &g, bool has_bn);
// BinActiv with q_k in place of sign(): kbits planes of index bits, [kbits][N][H][W][Cw].
cudaError_t launch_binactiv_kbit(const float *x, const float *scale, const float *shift,
                                 const ConvGeom &g, int kbits, uint32_t *x_planes, float *A, float *K,
                                 cudaStream_t st);
bool binconv_popc_supported(const ConvGeom &g);
cudaError_t launch_binconv_popc(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                                const float *K, const float *residual, const ConvGeom &g,
                                const EpiOpts &epi, float *out, int32_t *acc_out, cudaStream_t st);
// Function attributes (dynamic shared-memory limits) belong to a device: a launcher sets them
// once per device.  Returns the flag of the current device (out-of-range ids share the last).
inline bool &attr_done_for_current_device(bool (&flags)[64]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); dev = 0; }
  return flags[dev < 0 ? 0 : (dev > 63 ? 63 : dev)];
}

// Number of SMs of the current device, looked up once per device (persistent kernels size
// their grids by it).  148 if the query fails.
inline int sm_count_of_current_device() {
  static int counts[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 148; }
  const int slot = dev < 0 ? 0 : (dev > 63 ? 63 : dev);
  if (counts[slot] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = 148;
    }
    counts[slot] = n;
  }
  return counts[slot];
}

// Persistent tensor-core engine (strides 1 and 2).  Variants: one CTA per SM or CTA pairs
// (one MMA drives two SMs), each with the filters of a slab resident in shared memory when
// they fit or always streamed through a ring (re-expanded per work item).
enum TcVariant { kTcAuto = 0, kTcSingle, kTcSingleStream, kTcPair, kTcPairStream };
bool umma_tc_supported(const ConvGeom &g, TcVariant v);
cudaError_t launch_binconv_tc(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                              const float *K, const float *residual, const ConvGeom &g,
                              const EpiOpts &epi, float *out, int32_t *acc_out, TcVariant v,
                              cudaStream_t st);
// BinConv with the next layer's BinActiv fused into its epilogue (sign bits packed along the
// filters, partial sums of |y| per filter slab and epilogue warp); tc_fused_parts = number of
// partial planes for the shape (0: the fused kernel does not cover it).
int tc_fused_parts(const ConvGeom &g, TcVariant v);
cudaError_t launch_binconv_tc_fused(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                                    const float *K, const float *residual, const ConvGeom &g,
                                    float *out, const float *next_scale, const float *next_shift,
                                    uint32_t *xp_next, float *A_part, TcVariant v, cudaStream_t st);
// A = (sum of the partial planes) / C, then K = box filter of A for geometry g.
cudaError_t launch_binactiv_finish(const float *A_part, int parts, const ConvGeom &g, float *A,
                                   float *K, cudaStream_t st);
// Binary-Weight-Network convolution (Eq. 1) on bf16 activations laid out as a zero-padded pixel
// stream: elements of that stream for a geometry, its preparation from fp32 NCHW, the convolution.
bool bwn_supported(const ConvGeom &g);
size_t bwn_stream_elems(const ConvGeom &g);
cudaError_t launch_bwn_prepare(const float *x, const float *scale, const float *shift,
                               const ConvGeom &g, uint16_t *x_stream, cudaStream_t st);
cudaError_t launch_bwn_conv(const uint16_t *x_stream, const uint32_t *wp, const float *alpha,
                            const float *residual, const ConvGeom &g, float *out, cudaStream_t st);
cudaError_t read_status_bwn(int *status);
// Measured rates of the tensor pipe (1-bit MACs of the mxf4 MMA per clock per SM) and of the
// CUDA-core population count (popc per clock per SM) on the current device.  Synchronises.
cudaError_t measure_pipe_peaks(double *mma_mac_per_clk_per_sm, double *popc_per_clk_per_sm,
                               cudaStream_t st);
// A one-warp kernel whose bounded wait expires (nothing signals its barrier).
cudaError_t launch_wait_timeout_selftest(cudaStream_t st);
// Reads (and clears if set) the device status word of the tensor-core kernel.
cudaError_t read_status_tc(int *status);
// Same for the BinActiv kernel that waits on bulk copies.
cudaError_t read_status_act(int *status);
// Kernels launch_binactiv launches for this shape (1 or 2).
int binactiv_launch_count(const ConvGeom &g, bool has_bn);
cudaError_t launch_maxpool2d(const float *x, int N, int C, int H, int W, int k, int stride, int pad,
                             bool relu, float *out, cudaStream_t st);
cudaError_t launch_shortcut_conv1x1(const float *x, const float *w, int N, int C, int H, int W,
                                    int Co, int stride, float *out, cudaStream_t st);

}  // namespace xnor
