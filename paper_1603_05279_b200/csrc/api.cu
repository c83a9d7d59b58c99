// C-ABI entry points of libxnor: argument checks and dispatch.  No kernel code.
#include <atomic>

#include "bgrad.cuh"
#include "kbit.cuh"

namespace {

// The one piece of process-wide state: which BinConv engine the calls use.  An atomic, read
// once per call, so that a change from another thread is seen whole by the calls after it.
std::atomic<int> g_engine_state{(int)XNOR_ENGINE_AUTO};
inline xnor_engine current_engine() {
  return (xnor_engine)g_engine_state.load(std::memory_order_relaxed);
}

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }
inline bool bad_ptr(const void *p) { return p == nullptr || misaligned(p); }

xnor_status check_desc(const xnor_conv_desc *d, bool need_cout) {
  if (!d) return XNOR_ERR_INVALID_ARG;
  if (d->N <= 0 || d->C_in <= 0 || d->H <= 0 || d->W <= 0 || d->k_h <= 0 || d->k_w <= 0)
    return XNOR_ERR_INVALID_ARG;
  if (need_cout && d->C_out <= 0) return XNOR_ERR_INVALID_ARG;
  if (d->stride < 1 || d->pad < 0) return XNOR_ERR_INVALID_ARG;
  if (d->k_h > d->H + 2 * d->pad || d->k_w > d->W + 2 * d->pad) return XNOR_ERR_INVALID_ARG;
  if (d->flags & ~(XNOR_FLAG_RELU | XNOR_FLAG_K_VALID_TAPS)) return XNOR_ERR_INVALID_ARG;
  return XNOR_OK;
}

xnor_status from_cuda(cudaError_t e) { return e == cudaSuccess ? XNOR_OK : XNOR_ERR_CUDA; }

}  // namespace

extern "C" {

int xnor_version(void) { return 200; }

int xnor_built_with_bounds_check(void) {
#ifdef XNOR_BOUNDS_CHECK
  return 1;
#else
  return 0;
#endif
}

const char *xnor_status_string(xnor_status s) {
  switch (s) {
    case XNOR_OK: return "XNOR_OK";
    case XNOR_ERR_INVALID_ARG: return "XNOR_ERR_INVALID_ARG";
    case XNOR_ERR_UNSUPPORTED: return "XNOR_ERR_UNSUPPORTED";
    case XNOR_ERR_CUDA: return "XNOR_ERR_CUDA";
    case XNOR_ERR_TIMEOUT: return "XNOR_ERR_TIMEOUT";
    case XNOR_ERR_BOUNDS: return "XNOR_ERR_BOUNDS";
  }
  return "XNOR_ERR_UNKNOWN";
}

size_t xnor_words_per_pixel(int C_in) { return C_in > 0 ? (size_t)(C_in + 31) / 32 : 0; }

int xnor_out_extent(int in, int k, int stride, int pad) {
  if (in <= 0 || k <= 0 || stride < 1 || pad < 0 || k > in + 2 * pad) return 0;
  return (in + 2 * pad - k) / stride + 1;
}

xnor_status xnor_set_engine(xnor_engine e) {
  if ((int)e < (int)XNOR_ENGINE_AUTO || (int)e > (int)XNOR_ENGINE_UMMA_PAIR_STREAM)
    return XNOR_ERR_INVALID_ARG;
  g_engine_state.store((int)e, std::memory_order_relaxed);
  return XNOR_OK;
}

xnor_engine xnor_get_engine(void) { return current_engine(); }

xnor_status xnor_binarize_weights(const float *w, int C_out, int C_in, int k_h, int k_w,
                                  uint32_t *w_packed, float *alpha, void *cuda_stream) {
  if (bad_ptr(w) || bad_ptr(w_packed) || bad_ptr(alpha)) return XNOR_ERR_INVALID_ARG;
  if (C_out <= 0 || C_in <= 0 || k_h <= 0 || k_w <= 0) return XNOR_ERR_INVALID_ARG;
  if ((long long)k_h * k_w * ((C_in + 31) / 32) > 12288) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_binarize_weights(w, C_out, C_in, k_h, k_w, w_packed, alpha,
                                                 (cudaStream_t)cuda_stream));
}

xnor_status xnor_binactiv(const float *x, const float *bn_scale, const float *bn_shift,
                          const xnor_conv_desc *d, uint32_t *x_packed, float *A, float *K,
                          void *cuda_stream) {
  xnor_status s = check_desc(d, false);
  if (s != XNOR_OK) return s;
  if (bad_ptr(x) || bad_ptr(x_packed) || bad_ptr(A) || bad_ptr(K)) return XNOR_ERR_INVALID_ARG;
  if ((bn_scale == nullptr) != (bn_shift == nullptr)) return XNOR_ERR_INVALID_ARG;
  if (bn_scale && (misaligned(bn_scale) || misaligned(bn_shift))) return XNOR_ERR_INVALID_ARG;
  const xnor::ConvGeom g = xnor::make_geom(*d);
  if (!xnor::binactiv_supported(g, bn_scale != nullptr)) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_binactiv(x, bn_scale, bn_shift, g, x_packed, A, K,
                                         (cudaStream_t)cuda_stream));
}

xnor_status xnor_binactiv_static(const float *x, const float *bn_scale, const float *bn_shift,
                                 const xnor_conv_desc *d, uint32_t *x_packed, float *K,
                                 void *cuda_stream) {
  xnor_status s = check_desc(d, false);
  if (s != XNOR_OK) return s;
  if (bad_ptr(x) || bad_ptr(x_packed) || bad_ptr(K)) return XNOR_ERR_INVALID_ARG;
  if ((bn_scale == nullptr) != (bn_shift == nullptr)) return XNOR_ERR_INVALID_ARG;
  if (bn_scale && (misaligned(bn_scale) || misaligned(bn_shift))) return XNOR_ERR_INVALID_ARG;
  if ((unsigned long long)d->N * d->H * d->W > XNOR_BINACTIV_STATIC_MAX_PIXELS)
    return XNOR_ERR_UNSUPPORTED;
  const xnor::ConvGeom g = xnor::make_geom(*d);
  if (!xnor::binactiv_supported(g, bn_scale != nullptr)) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_binactiv_static(x, bn_scale, bn_shift, g, x_packed, K,
                                                (cudaStream_t)cuda_stream));
}

namespace {

xnor::TcVariant variant_of(xnor_engine e) {
  if (e == XNOR_ENGINE_UMMA_STREAM) return xnor::kTcSingleStream;
  if (e == XNOR_ENGINE_UMMA_SINGLE) return xnor::kTcSingle;
  if (e == XNOR_ENGINE_UMMA_PAIR) return xnor::kTcPair;
  if (e == XNOR_ENGINE_UMMA_PAIR_STREAM) return xnor::kTcPairStream;
  return xnor::kTcAuto;
}

// Which engine runs shape g under engine choice e: 1 tensor cores, 0 CUDA cores, -1 neither.
int pick_engine(const xnor::ConvGeom &g, xnor_engine e) {
  const bool tc_ok = e != XNOR_ENGINE_POPC && xnor::umma_tc_supported(g, variant_of(e));
  if (tc_ok) return 1;
  if (e != XNOR_ENGINE_AUTO && e != XNOR_ENGINE_POPC) return -1;
  return xnor::binconv_popc_supported(g) ? 0 : -1;
}

xnor_status check_conv_args(const uint32_t *x_packed, const uint32_t *w_packed, const float *alpha,
                            const float *K, const float *residual, const xnor_conv_desc *d,
                            const float *out, const int32_t *acc_out) {
  xnor_status s = check_desc(d, true);
  if (s != XNOR_OK) return s;
  if (bad_ptr(x_packed) || bad_ptr(w_packed) || bad_ptr(alpha) || bad_ptr(K) || bad_ptr(out))
    return XNOR_ERR_INVALID_ARG;
  if ((residual && misaligned(residual)) || (acc_out && misaligned(acc_out)))
    return XNOR_ERR_INVALID_ARG;
  if (d->k_h > 11 || d->k_w > 11) return XNOR_ERR_UNSUPPORTED;
  if ((long long)d->C_in * d->k_h * d->k_w >= (1LL << 24)) return XNOR_ERR_UNSUPPORTED;
  return XNOR_OK;
}

xnor_status run_conv(int engine, xnor_engine choice, const uint32_t *x_packed,
                     const uint32_t *w_packed, const float *alpha, const float *K,
                     const float *residual, const xnor::ConvGeom &g, const xnor::EpiOpts &epi,
                     float *out, int32_t *acc_out, cudaStream_t st) {
  if (engine == 1)
    return from_cuda(xnor::launch_binconv_tc(x_packed, w_packed, alpha, K, residual, g, epi, out,
                                             acc_out, variant_of(choice), st));
  return from_cuda(xnor::launch_binconv_popc(x_packed, w_packed, alpha, K, residual, g, epi, out,
                                             acc_out, st));
}

}  // namespace

xnor_status xnor_conv2d_forward(const uint32_t *x_packed, const uint32_t *w_packed,
                                const float *alpha, const float *K, const float *residual,
                                const xnor_conv_desc *d, float *out, int32_t *acc_out,
                                void *cuda_stream) {
  xnor_status s = check_conv_args(x_packed, w_packed, alpha, K, residual, d, out, acc_out);
  if (s != XNOR_OK) return s;
  const xnor::ConvGeom g = xnor::make_geom(*d);
  const xnor_engine choice = current_engine();
  const int engine = pick_engine(g, choice);
  if (engine < 0) return XNOR_ERR_UNSUPPORTED;
  return run_conv(engine, choice, x_packed, w_packed, alpha, K, residual, g, xnor::default_epi(g),
                  out, acc_out, (cudaStream_t)cuda_stream);
}

xnor_status xnor_binactiv_kbit(const float *x, const float *bn_scale, const float *bn_shift,
                               const xnor_conv_desc *d, int kbits, uint32_t *x_planes, float *A,
                               float *K, void *cuda_stream) {
  xnor_status s = check_desc(d, false);
  if (s != XNOR_OK) return s;
  if (kbits < 1 || kbits > 7) return XNOR_ERR_INVALID_ARG;
  if (bad_ptr(x) || bad_ptr(x_planes) || bad_ptr(A) || bad_ptr(K)) return XNOR_ERR_INVALID_ARG;
  if ((bn_scale == nullptr) != (bn_shift == nullptr)) return XNOR_ERR_INVALID_ARG;
  if (bn_scale && (misaligned(bn_scale) || misaligned(bn_shift))) return XNOR_ERR_INVALID_ARG;
  if (d->N > 65535) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_binactiv_kbit(x, bn_scale, bn_shift, xnor::make_geom(*d), kbits,
                                              x_planes, A, K, (cudaStream_t)cuda_stream));
}

xnor_status xnor_conv2d_forward_kbit(const uint32_t *x_planes, int kbits, const uint32_t *w_packed,
                                     const float *alpha, const float *K, const float *residual,
                                     const xnor_conv_desc *d, float *out, int32_t *acc_out,
                                     void *cuda_stream) {
  xnor_status s = check_conv_args(x_planes, w_packed, alpha, K, residual, d, out, acc_out);
  if (s != XNOR_OK) return s;
  if (kbits < 1 || kbits > 7) return XNOR_ERR_INVALID_ARG;
  const size_t plane_words = (size_t)d->N * d->H * d->W * ((d->C_in + 31) / 32);
  if (kbits > 1 && (plane_words & 3u)) return XNOR_ERR_UNSUPPORTED;   // planes stay 16-byte aligned
  const xnor::ConvGeom g = xnor::make_geom(*d);
  const xnor_engine choice = current_engine();
  const int engine = pick_engine(g, choice);
  if (engine < 0) return XNOR_ERR_UNSUPPORTED;
  // One pass per bit plane: with index bits b_p the level code is sum_p 2^p (2 b_p - 1), so the
  // sum over codes is sum_p 2^p (sum over plane p); pass p adds D_p K alpha 2^p / (2^k - 1) to
  // what the passes before it wrote (the output is its own residual).
  const double levels = (double)((1 << kbits) - 1);
  for (int p = 0; p < kbits; ++p) {
    xnor::EpiOpts epi = xnor::default_epi(g);
    epi.relu = epi.relu && p == kbits - 1;
    epi.out_scale = (float)((double)(1 << p) / levels);
    epi.acc_shift = p;
    epi.acc_accum = p > 0;
    s = run_conv(engine, choice, x_planes + (size_t)p * plane_words, w_packed, alpha, K,
                 p == 0 ? residual : out, g, epi, out, acc_out, (cudaStream_t)cuda_stream);
    if (s != XNOR_OK) return s;
  }
  return XNOR_OK;
}

namespace {

xnor::TcVariant current_variant() { return variant_of(current_engine()); }

bool good_desc(const xnor_conv_desc *d) {
  return d && d->N > 0 && d->C_in > 0 && d->H > 0 && d->W > 0 && d->C_out > 0 && d->k_h > 0 &&
         d->k_w > 0 && d->stride >= 1 && d->pad >= 0 && d->k_h <= d->H + 2 * d->pad &&
         d->k_w <= d->W + 2 * d->pad && !(d->flags & ~(XNOR_FLAG_RELU | XNOR_FLAG_K_VALID_TAPS));
}

}  // namespace

int xnor_binactiv_launches(const xnor_conv_desc *d, int has_bn) {
  if (!good_desc(d)) return 0;
  const xnor::ConvGeom g = xnor::make_geom(*d);
  if (!xnor::binactiv_supported(g, has_bn != 0)) return 0;
  return xnor::binactiv_launch_count(g, has_bn != 0);
}

int xnor_binactiv_kbit_launches(const xnor_conv_desc *d, int kbits, int has_bn) {
  if (!good_desc(d) || kbits < 1 || kbits > 7) return 0;
  return xnor::binactiv_kbit_launch_count(xnor::make_geom(*d), has_bn != 0, kbits);
}

int xnor_conv2d_binactiv_parts(const xnor_conv_desc *d) {
  if (!good_desc(d) || current_engine() == XNOR_ENGINE_POPC || d->k_h > 11 || d->k_w > 11 ||
      (long long)d->C_in * d->k_h * d->k_w >= (1LL << 24))
    return 0;
  return xnor::tc_fused_parts(xnor::make_geom(*d), current_variant());
}

xnor_status xnor_conv2d_forward_binactiv(const uint32_t *x_packed, const uint32_t *w_packed,
                                         const float *alpha, const float *K, const float *residual,
                                         const xnor_conv_desc *d, float *out, const float *next_scale,
                                         const float *next_shift, uint32_t *x_packed_next,
                                         float *A_parts, void *cuda_stream) {
  if (!good_desc(d)) return XNOR_ERR_INVALID_ARG;
  if (bad_ptr(x_packed) || bad_ptr(w_packed) || bad_ptr(alpha) || bad_ptr(K) ||
      bad_ptr(x_packed_next) || bad_ptr(A_parts))
    return XNOR_ERR_INVALID_ARG;
  if ((residual && misaligned(residual)) || (out && misaligned(out)) ||
      (next_scale == nullptr) != (next_shift == nullptr) ||
      (next_scale && (misaligned(next_scale) || misaligned(next_shift))))
    return XNOR_ERR_INVALID_ARG;
  if (xnor_conv2d_binactiv_parts(d) == 0) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_binconv_tc_fused(x_packed, w_packed, alpha, K, residual,
                                                 xnor::make_geom(*d), out, next_scale, next_shift,
                                                 x_packed_next, A_parts, current_variant(),
                                                 (cudaStream_t)cuda_stream));
}

xnor_status xnor_binactiv_finish(const float *A_parts, int parts, const xnor_conv_desc *d_next,
                                 float *A, float *K, void *cuda_stream) {
  if (!good_desc(d_next) || parts < 1 || bad_ptr(A_parts) || bad_ptr(A) || bad_ptr(K))
    return XNOR_ERR_INVALID_ARG;
  if (d_next->N > 65535) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_binactiv_finish(A_parts, parts, xnor::make_geom(*d_next), A, K,
                                                (cudaStream_t)cuda_stream));
}

xnor_status xnor_maxpool2d(const float *x, int N, int C, int H, int W, int k, int stride, int pad,
                           int relu, float *out, void *cuda_stream) {
  if (bad_ptr(x) || bad_ptr(out)) return XNOR_ERR_INVALID_ARG;
  if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || k < 1 || stride < 1 || pad < 0 || pad >= k ||
      k > H + 2 * pad || k > W + 2 * pad)
    return XNOR_ERR_INVALID_ARG;
  if (k > 11) return XNOR_ERR_UNSUPPORTED;
  if ((long long)((H + 2 * pad - k) / stride + 1) * ((W + 2 * pad - k) / stride + 1) >= (1ll << 30))
    return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_maxpool2d(x, N, C, H, W, k, stride, pad, relu != 0, out,
                                          (cudaStream_t)cuda_stream));
}

xnor_status xnor_selftest_wait_timeout(void *cuda_stream) {
  return from_cuda(xnor::launch_wait_timeout_selftest((cudaStream_t)cuda_stream));
}

xnor_status xnor_check_device(void *cuda_stream) {
  int st = 0, st2 = 0, st3 = 0;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess ||
      xnor::read_status_tc(&st) != cudaSuccess || xnor::read_status_bwn(&st2) != cudaSuccess ||
      xnor::read_status_act(&st3) != cudaSuccess) {
    (void)cudaGetLastError();
    return XNOR_ERR_CUDA;
  }
  if (st >= 1000) return XNOR_ERR_BOUNDS;
  return (st == 0 && st2 == 0 && st3 == 0) ? XNOR_OK : XNOR_ERR_TIMEOUT;
}

xnor_status xnor_measure_peaks(double *mma_mac_per_clk_per_sm, double *popc_per_clk_per_sm,
                               void *cuda_stream) {
  if (mma_mac_per_clk_per_sm == nullptr || popc_per_clk_per_sm == nullptr) return XNOR_ERR_INVALID_ARG;
  const cudaError_t e = xnor::measure_pipe_peaks(mma_mac_per_clk_per_sm, popc_per_clk_per_sm,
                                                 (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) (void)cudaGetLastError();
  return from_cuda(e);
}

size_t xnor_bwn_input_elems(const xnor_conv_desc *d) {
  if (!good_desc(d)) return 0;
  return xnor::bwn_stream_elems(xnor::make_geom(*d));
}

xnor_status xnor_bwn_prepare_input(const float *x, const float *bn_scale, const float *bn_shift,
                                   const xnor_conv_desc *d, uint16_t *x_stream, void *cuda_stream) {
  if (!good_desc(d)) return XNOR_ERR_INVALID_ARG;
  if (bad_ptr(x) || bad_ptr(x_stream)) return XNOR_ERR_INVALID_ARG;
  if ((bn_scale == nullptr) != (bn_shift == nullptr)) return XNOR_ERR_INVALID_ARG;
  if (bn_scale && (misaligned(bn_scale) || misaligned(bn_shift))) return XNOR_ERR_INVALID_ARG;
  const xnor::ConvGeom g = xnor::make_geom(*d);
  if (!xnor::bwn_supported(g)) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_bwn_prepare(x, bn_scale, bn_shift, g, x_stream,
                                            (cudaStream_t)cuda_stream));
}

xnor_status xnor_bwn_conv2d_forward(const uint16_t *x_stream, const uint32_t *w_packed,
                                    const float *alpha, const float *residual,
                                    const xnor_conv_desc *d, float *out, void *cuda_stream) {
  if (!good_desc(d)) return XNOR_ERR_INVALID_ARG;
  if (bad_ptr(x_stream) || bad_ptr(w_packed) || bad_ptr(alpha) || bad_ptr(out) ||
      (residual && misaligned(residual)))
    return XNOR_ERR_INVALID_ARG;
  const xnor::ConvGeom g = xnor::make_geom(*d);
  if (!xnor::bwn_supported(g)) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_bwn_conv(x_stream, w_packed, alpha, residual, g, out,
                                         (cudaStream_t)cuda_stream));
}

namespace {

// Geometry of the backward convolution of the forward layer d: the gradient
// [C_out][H_out][W_out] convolved at stride 1 with pad k - 1 - pad gives [C_in][H][W].
bool backward_geom(const xnor_conv_desc *d, xnor::ConvGeom *gb) {
  if (!good_desc(d) || d->stride != 1 || d->k_h != d->k_w || d->N > 65535) return false;
  const xnor::ConvGeom g = xnor::make_geom(*d);
  xnor_conv_desc b = *d;
  b.C_in = d->C_out; b.C_out = d->C_in; b.H = g.Ho; b.W = g.Wo;
  b.pad = d->k_h - 1 - d->pad; b.flags = 0;
  *gb = xnor::make_geom(b);
  return gb->Ho == d->H && gb->Wo == d->W && xnor::bwn_supported(*gb);
}

}  // namespace

size_t xnor_bgrad_stream_elems(const xnor_conv_desc *d) {
  xnor::ConvGeom gb;
  return backward_geom(d, &gb) ? xnor::bwn_stream_elems(gb) : 0;
}

xnor_status xnor_binarize_weights_transposed(const float *w, int C_out, int C_in, int k_h, int k_w,
                                             uint32_t *wT_packed, void *cuda_stream) {
  if (bad_ptr(w) || bad_ptr(wT_packed)) return XNOR_ERR_INVALID_ARG;
  if (C_out <= 0 || C_in <= 0 || k_h <= 0 || k_w <= 0) return XNOR_ERR_INVALID_ARG;
  if ((long long)k_h * k_w * ((C_out + 31) / 32) > 12288) return XNOR_ERR_UNSUPPORTED;
  return from_cuda(xnor::launch_binarize_weights_transposed(w, C_out, C_in, k_h, k_w, wT_packed,
                                                            (cudaStream_t)cuda_stream));
}

xnor_status xnor_binary_gradient_backward(const float *g, const uint32_t *wT_packed,
                                          const float *alpha, const xnor_conv_desc *d, float *gmax,
                                          uint16_t *g_stream, float *grad_in, void *cuda_stream) {
  if (!good_desc(d)) return XNOR_ERR_INVALID_ARG;
  if (bad_ptr(g) || bad_ptr(wT_packed) || bad_ptr(alpha) || bad_ptr(gmax) || bad_ptr(g_stream) ||
      bad_ptr(grad_in))
    return XNOR_ERR_INVALID_ARG;
  xnor::ConvGeom gb;
  if (!backward_geom(d, &gb)) return XNOR_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  cudaError_t e = xnor::launch_grad_max(g, gb.N, (size_t)gb.C * gb.H * gb.W, gmax, st);
  if (e == cudaSuccess) e = xnor::launch_bwn_prepare_grad(g, alpha, gmax, gb, g_stream, st);
  if (e == cudaSuccess) e = xnor::launch_bwn_conv(g_stream, wT_packed, nullptr, nullptr, gb, grad_in, st);
  if (e != cudaSuccess) (void)cudaGetLastError();
  return from_cuda(e);
}

xnor_status xnor_shortcut_conv1x1(const float *x, const float *w, int N, int C_in, int H, int W,
                                  int C_out, int stride, float *out, void *cuda_stream) {
  if (bad_ptr(x) || bad_ptr(w) || bad_ptr(out)) return XNOR_ERR_INVALID_ARG;
  if (N <= 0 || C_in <= 0 || H <= 0 || W <= 0 || C_out <= 0 || stride < 1)
    return XNOR_ERR_INVALID_ARG;
  return from_cuda(xnor::launch_shortcut_conv1x1(x, w, N, C_in, H, W, C_out, stride, out,
                                                 (cudaStream_t)cuda_stream));
}

}  // extern "C"
