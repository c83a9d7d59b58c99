/*
 * CPU oracle for the XNOR-Net binary-convolution forward block
 * (BatchNorm affine -> BinActiv -> BinConv), arxiv 1603.05279.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain, nested-loop
 * statement of what the block computes, written from the paper's equations in
 * +/-1 arithmetic: no bit packing, no popcount, no tiling, no fusion.  Only the
 * test-suite, the smoke check and the CPU-baseline leg of the benchmark may
 * call it; the CUDA library never does, and the two share no code.
 *
 * Conventions (one reading of each point the paper leaves open):
 *   - tensors are dense row-major: x[N][C][H][W], w[Co][C][kh][kw],
 *     out[N][Co][Ho][Wo], Ho = (H + 2*pad - kh)/stride + 1 (same for Wo);
 *   - sign(v) = +1 when v >= 0 (so +0 and -0 give +1), else -1
 *     (Section 3.1, the assignment below Eq. 4; used for inputs too);
 *   - the BN affine is ONE fused multiply-add in fp32, y = fmaf(scale,x,shift);
 *   - zero padding: a tap that falls outside the image contributes 0 to the
 *     binary convolution and 0 to the box filter that makes K; the box filter
 *     always divides by kh*kw (K = A * k with k_ij = 1/(w h), Section 3.2);
 *   - real-valued sums (alpha, A, K, out) are accumulated in double and
 *     rounded to float once; the +/-1 convolution is exact int32.
 *
 * Options beyond the main path (each a function of its own further down, all
 * pinned by the CPU tests): the border variant of K that divides by the taps
 * inside the image, ReLU on the block's output, k-bit activations q_k in place
 * of sign(), the Binary-Weight-Network convolution of Eq. 1 on real inputs, and
 * the backward convolution with a binarised gradient.
 *
 * The only parallelism is an OpenMP "parallel for" over independent outer
 * indices (images, filters); loop bodies are unchanged by it.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

static int out_extent(int in, int k, int stride, int pad) {
  return (in + 2 * pad - k) / stride + 1;
}

/* Block order B-A-C-P, Section 3.2 "Training XNOR-Networks": the input is
 * normalised before it is binarised.  At inference BatchNorm is a per-channel
 * affine map; scale and shift are inputs (folded by the caller).
 * scale == NULL means identity (y = x). */
void oracle_bn_affine(const float *x, const float *scale, const float *shift,
                      int N, int C, int H, int W, float *y) {
  const size_t hw = (size_t)H * W;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int c = 0; c < C; ++c) {
      const float *xp = x + ((size_t)n * C + c) * hw;
      float *yp = y + ((size_t)n * C + c) * hw;
      for (size_t i = 0; i < hw; ++i)
        yp[i] = scale ? fmaf(scale[c], xp[i], shift[c]) : xp[i];
    }
}

/* sign() of Eq. 4 / Eq. 9: +1 for v >= 0, -1 otherwise, as int8. */
void oracle_sign(const float *v, size_t count, int8_t *s) {
#pragma omp parallel for schedule(static)
  for (size_t i = 0; i < count; ++i) s[i] = (v[i] >= 0.0f) ? 1 : -1;
}

/* Section 3.2 "Binary Convolution": A = (sum over channels of |I|) / c,
 * one value per spatial position of each image. */
void oracle_channel_abs_mean(const float *y, int N, int C, int H, int W,
                             float *A) {
  const size_t hw = (size_t)H * W;
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n)
    for (size_t i = 0; i < hw; ++i) {
      double s = 0.0;
      for (int c = 0; c < C; ++c) s += fabs((double)y[((size_t)n * C + c) * hw + i]);
      A[(size_t)n * hw + i] = (float)(s / (double)C);
    }
}

/* Section 3.2: K = A * k, k a kh x kw filter whose entries are all
 * 1/(kh*kw); evaluated at the convolution's own output positions (same
 * stride and zero padding), so K[n][oy][ox] is the scale beta of the input
 * window that output (oy,ox) sees. */
void oracle_box_filter(const float *A, int N, int H, int W, int kh, int kw,
                       int stride, int pad, float *K) {
  const int Ho = out_extent(H, kh, stride, pad), Wo = out_extent(W, kw, stride, pad);
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n)
    for (int oy = 0; oy < Ho; ++oy)
      for (int ox = 0; ox < Wo; ++ox) {
        double s = 0.0;
        for (int ky = 0; ky < kh; ++ky)
          for (int kx = 0; kx < kw; ++kx) {
            const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
            if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue; /* pad adds 0 */
            s += (double)A[((size_t)n * H + iy) * W + ix];
          }
        K[((size_t)n * Ho + oy) * Wo + ox] = (float)(s / (double)(kh * kw));
      }
}

/* Eq. 4 and Eq. 6 (also Algorithm 1, the two assignments inside the filter
 * loop): per filter, B = sign(W) and alpha = ||W||_1 / n, n = c*kh*kw. */
void oracle_binarize_weights(const float *w, int Co, int C, int kh, int kw,
                             int8_t *B, float *alpha) {
  const size_t n = (size_t)C * kh * kw;
#pragma omp parallel for schedule(static)
  for (int co = 0; co < Co; ++co) {
    double l1 = 0.0;
    for (size_t i = 0; i < n; ++i) {
      const float v = w[(size_t)co * n + i];
      B[(size_t)co * n + i] = (v >= 0.0f) ? 1 : -1;
      l1 += fabs((double)v);
    }
    alpha[co] = (float)(l1 / (double)n);
  }
}

/* The binary convolution sign(I) (*) sign(W) of Eq. 11, written as the sum of
 * products of +/-1 values that XNOR + bitcount evaluates (Section 3.2, first
 * paragraph).  Taps outside the image add nothing. */
void oracle_binconv_acc(const int8_t *Hs, const int8_t *B, int N, int C, int H,
                        int W, int Co, int kh, int kw, int stride, int pad,
                        int32_t *acc) {
  const int Ho = out_extent(H, kh, stride, pad), Wo = out_extent(W, kw, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < Co; ++co)
      for (int oy = 0; oy < Ho; ++oy)
        for (int ox = 0; ox < Wo; ++ox) {
          int32_t s = 0;
          for (int c = 0; c < C; ++c)
            for (int ky = 0; ky < kh; ++ky)
              for (int kx = 0; kx < kw; ++kx) {
                const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
                if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue;
                s += (int32_t)Hs[(((size_t)n * C + c) * H + iy) * W + ix] *
                     (int32_t)B[(((size_t)co * C + c) * kh + ky) * kw + kx];
              }
          acc[(((size_t)n * Co + co) * Ho + oy) * Wo + ox] = s;
        }
}

/* The "(.) K alpha" of Eq. 11: K is per image and position, shared by all
 * filters; alpha is per filter.  residual (nullable) is added afterwards
 * (ResNet shortcut). */
void oracle_scale_output(const int32_t *acc, const float *K, const float *alpha,
                         const float *residual, int N, int Co, int Ho, int Wo,
                         float *out) {
  const size_t hw = (size_t)Ho * Wo;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < Co; ++co)
      for (size_t i = 0; i < hw; ++i) {
        const size_t o = ((size_t)n * Co + co) * hw + i;
        double v = (double)acc[o] * (double)K[(size_t)n * hw + i] * (double)alpha[co];
        if (residual) v += (double)residual[o];
        out[o] = (float)v;
      }
}

/* Whole block in the paper's order: BN -> BinActiv (sign, A, K) -> BinConv.
 * Every intermediate is returned so each can be compared on its own.
 * Buffers (caller-allocated): y[N*C*H*W] float, Hs[N*C*H*W] int8,
 * A[N*H*W], K[N*Ho*Wo], B[Co*C*kh*kw] int8, alpha[Co],
 * acc[N*Co*Ho*Wo] int32, out[N*Co*Ho*Wo]. */
void oracle_xnor_block(const float *x, const float *bn_scale, const float *bn_shift,
                       const float *w, const float *residual, int N, int C, int H,
                       int W, int Co, int kh, int kw, int stride, int pad,
                       float *y, int8_t *Hs, float *A, float *K, int8_t *B,
                       float *alpha, int32_t *acc, float *out) {
  const int Ho = out_extent(H, kh, stride, pad), Wo = out_extent(W, kw, stride, pad);
  oracle_bn_affine(x, bn_scale, bn_shift, N, C, H, W, y);
  oracle_sign(y, (size_t)N * C * H * W, Hs);
  oracle_channel_abs_mean(y, N, C, H, W, A);
  oracle_box_filter(A, N, H, W, kh, kw, stride, pad, K);
  oracle_binarize_weights(w, Co, C, kh, kw, B, alpha);
  oracle_binconv_acc(Hs, B, N, C, H, W, Co, kh, kw, stride, pad, acc);
  oracle_scale_output(acc, K, alpha, residual, N, Co, Ho, Wo, out);
}

/* The same block with the options the paper mentions around it: kbits > 1
 * quantises the normalised input with q_k instead of sign() (Hs then holds the
 * level codes, and the sums are divided by 2^k - 1); k_valid_taps selects the
 * border variant of K; relu applies max(., 0) to the block's output.  With
 * kbits = 1 and both flags 0 it is oracle_xnor_block.  Forward declarations:
 * the option functions are defined further down. */
void oracle_box_filter_valid_taps(const float *A, int N, int H, int W, int kh, int kw,
                                  int stride, int pad, float *K);
void oracle_relu(float *v, size_t count);
void oracle_quantize_k(const float *v, size_t count, int k, int8_t *L);
void oracle_scale_output_k(const int32_t *acc, int k, const float *K, const float *alpha,
                           const float *residual, int N, int Co, int Ho, int Wo, float *out);

void oracle_xnor_block_ex(const float *x, const float *bn_scale, const float *bn_shift,
                          const float *w, const float *residual, int N, int C, int H,
                          int W, int Co, int kh, int kw, int stride, int pad, int kbits,
                          int relu, int k_valid_taps, float *y, int8_t *Hs, float *A,
                          float *K, int8_t *B, float *alpha, int32_t *acc, float *out) {
  const int Ho = out_extent(H, kh, stride, pad), Wo = out_extent(W, kw, stride, pad);
  oracle_bn_affine(x, bn_scale, bn_shift, N, C, H, W, y);
  if (kbits == 1) oracle_sign(y, (size_t)N * C * H * W, Hs);
  else oracle_quantize_k(y, (size_t)N * C * H * W, kbits, Hs);
  oracle_channel_abs_mean(y, N, C, H, W, A);
  if (k_valid_taps) oracle_box_filter_valid_taps(A, N, H, W, kh, kw, stride, pad, K);
  else oracle_box_filter(A, N, H, W, kh, kw, stride, pad, K);
  oracle_binarize_weights(w, Co, C, kh, kw, B, alpha);
  oracle_binconv_acc(Hs, B, N, C, H, W, Co, kh, kw, stride, pad, acc);
  if (kbits == 1) oracle_scale_output(acc, K, alpha, residual, N, Co, Ho, Wo, out);
  else oracle_scale_output_k(acc, kbits, K, alpha, residual, N, Co, Ho, Wo, out);
  if (relu) oracle_relu(out, (size_t)N * Co * Ho * Wo);
}

/* Full-precision 1x1 strided convolution without bias: the projection
 * shortcut ("type B") of the ResNet-18 variant in Section 4.2.  Plain
 * definition, double accumulation. */
void oracle_shortcut_conv1x1(const float *x, const float *w, int N, int C, int H,
                             int W, int Co, int stride, float *out) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < Co; ++co)
      for (int oy = 0; oy < Ho; ++oy)
        for (int ox = 0; ox < Wo; ++ox) {
          double s = 0.0;
          for (int c = 0; c < C; ++c)
            s += (double)x[(((size_t)n * C + c) * H + (size_t)oy * stride) * W + (size_t)ox * stride] *
                 (double)w[(size_t)co * C + c];
          out[(((size_t)n * Co + co) * Ho + oy) * Wo + ox] = (float)s;
        }
}

/* The last layer of the block of Section 3.2 ("Training XNOR-Networks": the
 * order is BatchNorm, BinActiv, BinConv, Pool, with an optional non-binary
 * activation such as ReLU after the binary convolution): max pooling over
 * k x k windows at the given stride, on the real-valued output of BinConv.
 * Readings where the paper is silent: a tap outside the image does not take
 * part in the maximum (at least one tap is always inside since pad < k);
 * Ho = (H + 2 pad - k) / stride + 1, rounded down; relu != 0 applies
 * max(v, 0) to every input value before the maximum. */
void oracle_maxpool2d(const float *x, int N, int C, int H, int W, int k, int stride,
                      int pad, int relu, float *out) {
  const int Ho = out_extent(H, k, stride, pad), Wo = out_extent(W, k, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int c = 0; c < C; ++c)
      for (int oy = 0; oy < Ho; ++oy)
        for (int ox = 0; ox < Wo; ++ox) {
          int first = 1;
          float m = 0.0f;
          for (int ky = 0; ky < k; ++ky)
            for (int kx = 0; kx < k; ++kx) {
              const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
              if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue;
              float v = x[(((size_t)n * C + c) * H + iy) * W + ix];
              if (relu && v < 0.0f) v = 0.0f;
              if (first || v > m) { m = v; first = 0; }
            }
          out[(((size_t)n * C + c) * Ho + oy) * Wo + ox] = m;
        }
}

/* Variant of the box filter for the border: the paper writes K = A * k without
 * saying how A is padded.  The main reading (oracle_box_filter) pads with zeros
 * and always divides by kh*kw.  This one averages over the taps that lie
 * inside the image only (divisor = their number), so that K is the mean of |I|
 * over exactly the input values the window sees; in the interior the two agree. */
void oracle_box_filter_valid_taps(const float *A, int N, int H, int W, int kh, int kw,
                                  int stride, int pad, float *K) {
  const int Ho = out_extent(H, kh, stride, pad), Wo = out_extent(W, kw, stride, pad);
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n)
    for (int oy = 0; oy < Ho; ++oy)
      for (int ox = 0; ox < Wo; ++ox) {
        double s = 0.0;
        int count = 0;
        for (int ky = 0; ky < kh; ++ky)
          for (int kx = 0; kx < kw; ++kx) {
            const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
            if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue;
            s += (double)A[((size_t)n * H + iy) * W + ix];
            ++count;
          }
        /* a window wholly inside the padding sees nothing: K = 0 there */
        K[((size_t)n * Ho + oy) * Wo + ox] = count ? (float)(s / (double)count) : 0.0f;
      }
}

/* Section 3.2, "Training XNOR-Networks": a non-binary activation such as ReLU
 * may follow the binary convolution.  Reading: it is applied to the value the
 * block writes, i.e. after the scaling by K alpha and after the shortcut add
 * where there is one.  In place on fp32 values (max with 0 is exact). */
void oracle_relu(float *v, size_t count) {
#pragma omp parallel for schedule(static)
  for (size_t i = 0; i < count; ++i)
    if (!(v[i] > 0.0f)) v[i] = (v[i] != v[i]) ? v[i] : 0.0f; /* NaN stays NaN */
}

/* Section 3.2, "k-bit Quantization": q_k(x) = 2([(2^k-1)(x+1)/2]/(2^k-1) - 1/2)
 * replaces sign(); [.] rounds to the nearest integer and x lies in [-1, 1].
 * The result is one of 2^k evenly spaced levels; written as an odd integer
 * code L = 2 i - (2^k - 1), i = [.] in 0 .. 2^k - 1, the level is L/(2^k - 1).
 * Readings: values outside [-1, 1] are clipped first; ties round up, which
 * makes k = 1 the sign() of Eq. 4 (+1 at zero).  The rounding decision is
 * taken in fp32, the precision of the data: [t] >= j exactly when
 * x >= tau_j = (2j - 1)/(2^k - 1) - 1, and x is compared with tau_j rounded to
 * float (tau_1 = 0 for k = 1).  1 <= k <= 7 (codes fit int8). */
void oracle_quantize_k(const float *v, size_t count, int k, int8_t *L) {
  const int levels = (1 << k) - 1; /* 2^k - 1 */
#pragma omp parallel for schedule(static)
  for (size_t i = 0; i < count; ++i) {
    float x = v[i];
    if (x > 1.0f) x = 1.0f;
    if (x < -1.0f) x = -1.0f;
    int idx = 0;
    for (int j = 1; j <= levels; ++j) {
      const float tau = (float)((double)(2 * j - 1) / (double)levels - 1.0);
      if (x >= tau) idx = j;
    }
    L[i] = (int8_t)(2 * idx - levels);
  }
}

/* Eq. 11 with q_k in place of sign(I): the integer sums of
 * oracle_binconv_acc over level codes are sums of L * (+-1); dividing by
 * 2^k - 1 turns codes into levels.  K, alpha and the residual as in
 * oracle_scale_output. */
void oracle_scale_output_k(const int32_t *acc, int k, const float *K, const float *alpha,
                           const float *residual, int N, int Co, int Ho, int Wo,
                           float *out) {
  const size_t hw = (size_t)Ho * Wo;
  const double levels = (double)((1 << k) - 1);
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < Co; ++co)
      for (size_t i = 0; i < hw; ++i) {
        const size_t o = ((size_t)n * Co + co) * hw + i;
        double v = (double)acc[o] / levels * (double)K[(size_t)n * hw + i] * (double)alpha[co];
        if (residual) v += (double)residual[o];
        out[o] = (float)v;
      }
}

/* Rounds fp32 values to bfloat16 (8 significand bits, round to nearest, ties
 * to even) and returns them as fp32: the activation format of the
 * Binary-Weight-Network convolution below.  Written on the bit pattern:
 * keep the upper 16 bits, round on the lower 16.  NaN and infinity pass. */
void oracle_round_bf16(const float *v, size_t count, float *r) {
  for (size_t i = 0; i < count; ++i) {
    union { float f; uint32_t u; } a;
    a.f = v[i];
    if ((a.u & 0x7F800000u) != 0x7F800000u) {
      const uint32_t lower = a.u & 0xFFFFu, upper = a.u >> 16;
      uint32_t up = upper;
      if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) up = upper + 1u;
      a.u = up << 16;
    }
    r[i] = a.f;
  }
}

/* Binary-Weight-Network convolution, Section 3.1, Eq. 1:
 * I * W ~ (I (+) B) alpha, where (+) is a convolution that only adds and
 * subtracts the real-valued inputs according to B = sign(W), and alpha is the
 * filter's scale (Eq. 6).  x holds the real inputs (the caller rounds them to
 * the format the convolution consumes), B and alpha come from
 * oracle_binarize_weights.  Zero padding; residual (nullable) added last. */
void oracle_bwn_conv(const float *x, const int8_t *B, const float *alpha,
                     const float *residual, int N, int C, int H, int W, int Co, int kh,
                     int kw, int stride, int pad, float *out) {
  const int Ho = out_extent(H, kh, stride, pad), Wo = out_extent(W, kw, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < Co; ++co)
      for (int oy = 0; oy < Ho; ++oy)
        for (int ox = 0; ox < Wo; ++ox) {
          double s = 0.0;
          for (int c = 0; c < C; ++c)
            for (int ky = 0; ky < kh; ++ky)
              for (int kx = 0; kx < kw; ++kx) {
                const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
                if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue;
                const double xv = (double)x[(((size_t)n * C + c) * H + iy) * W + ix];
                if (B[(((size_t)co * C + c) * kh + ky) * kw + kx] > 0) s += xv;
                else s -= xv;
              }
          const size_t o = (((size_t)n * Co + co) * Ho + oy) * Wo + ox;
          double v = s * (double)alpha[co];
          if (residual) v += (double)residual[o];
          out[o] = (float)v;
        }
}

/* Binary-gradient backward convolution, Section 3.2, "Binary Gradient".
 * The backward pass of a layer convolves the gradient g that arrives at the
 * convolution's output with the weight filters; as in Algorithm 1 the filters
 * are the binarised ones, alpha * sign(W).  The gradient is binarised the way
 * the forward operands are, sign(g), but scaled by max_i |g_i| instead of the
 * mean of Eq. 6.  Readings where the paragraph is silent: the maximum is taken
 * over one image's gradient tensor [Co][Ho][Wo] (images stay independent);
 * sign(0) = +1 as everywhere; stride 1, zero padding.  Result: the gradient with
 * respect to the convolution's input,
 *   gin[n][c][y][x] = sum_{co,ky,kx} alpha[co] B[co][c][ky][kx] gmax[n]
 *                                    sign(g[n][co][y + pad - ky][x + pad - kx]),
 * taps outside the gradient's extent contributing 0.
 * round_products != 0: every product gmax[n] * alpha[co] is formed in fp32 and
 * rounded to bfloat16 before it enters the sum (the operand format of the
 * tensor-core convolution that the library runs this on). */
void oracle_binary_gradient_backward(const float *g, const int8_t *B, const float *alpha, int N,
                                     int C, int H, int W, int Co, int kh, int kw, int pad,
                                     int round_products, float *gmax, float *gin) {
  const int Ho = out_extent(H, kh, 1, pad), Wo = out_extent(W, kw, 1, pad);
  const size_t per_image = (size_t)Co * Ho * Wo;
  for (int n = 0; n < N; ++n) {
    float m = 0.0f;
    for (size_t i = 0; i < per_image; ++i) {
      const float a = fabsf(g[(size_t)n * per_image + i]);
      if (a > m) m = a;
    }
    gmax[n] = m;
  }
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int c = 0; c < C; ++c)
      for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x) {
          double s = 0.0;
          for (int co = 0; co < Co; ++co) {
            float t = gmax[n] * alpha[co];
            if (round_products) oracle_round_bf16(&t, 1, &t);
            for (int ky = 0; ky < kh; ++ky)
              for (int kx = 0; kx < kw; ++kx) {
                const int oy = y + pad - ky, ox = x + pad - kx;
                if (oy < 0 || oy >= Ho || ox < 0 || ox >= Wo) continue;
                const float gv = g[(((size_t)n * Co + co) * Ho + oy) * Wo + ox];
                const int sg = gv >= 0.0f ? 1 : -1;
                const int b = B[(((size_t)co * C + c) * kh + ky) * kw + kx] > 0 ? 1 : -1;
                if (sg * b > 0) s += (double)t;
                else s -= (double)t;
              }
          }
          gin[(((size_t)n * C + c) * H + y) * W + x] = (float)s;
        }
}

/* Section 4.1: with 64 binary operations per clock, the ratio of the cost of
 * a standard convolution (c*N_W*N_I operations) to the binary one
 * (c*N_W*N_I/64 + N_I) is S = 64 c N_W / (c N_W + 64). */
double oracle_speedup_model(double c, double n_w) {
  return 64.0 * c * n_w / (c * n_w + 64.0);
}
