/*
 * libxnor -- forward path of the XNOR-Net binary convolution block
 * (BatchNorm affine -> BinActiv -> BinConv, arxiv 1603.05279) on one
 * NVIDIA B200 (sm_100a).
 *
 * Conventions shared by every call
 * --------------------------------
 *  - Every data pointer is a DEVICE pointer owned by the caller; the library
 *    allocates nothing and frees nothing.  Descriptor structs are read on the
 *    host during the call and need not outlive it.
 *  - Every pointer must be 16-byte aligned.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*,
 *    NULL = the legacy default stream) and return without synchronising.
 *    Outputs are fully overwritten.
 *  - Errors are returned as xnor_status; nothing is printed, thrown or
 *    aborted.  On any status other than XNOR_OK nothing was launched.
 *  - Tensors are dense, row-major, fp32 unless stated:
 *      activations  x  [N][C_in][H][W]               ("NCHW")
 *      filters      w  [C_out][C_in][k_h][k_w]       (no bias; the paper
 *                                                     assumes bias-free filters,
 *                                                     footnote in Section 3)
 *      output      out [N][C_out][H_out][W_out],
 *      H_out = (H + 2*pad - k_h)/stride + 1, likewise W_out.
 *  - sign(v) = +1 when v >= 0 (+0 and -0 included), -1 otherwise (the
 *    assignment under Eq. 4, used for weights and inputs alike).  A set bit
 *    means +1.
 *  - Bit packing is along channels in 32-bit words: channel c is bit (c % 32)
 *    of word (c / 32); Cw = ceil(C_in / 32) words per pixel or filter tap;
 *    unused high bits of the last word are 0 in both operands.  Activation
 *    words are pixel-major ([N][H][W][Cw]); filter words are stored in the
 *    order xnor_binarize_weights documents.
 *  - Zero padding: a filter tap that falls outside the image contributes 0 to
 *    the binary convolution and 0 to the box filter that makes K.
 */
#ifndef XNOR_H_
#define XNOR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  XNOR_OK = 0,
  XNOR_ERR_INVALID_ARG = 1, /* null/misaligned pointer, non-positive size, k > H + 2 pad ... */
  XNOR_ERR_UNSUPPORTED = 2, /* a shape the kernels were not built for (see each call)       */
  XNOR_ERR_CUDA = 3,        /* the launch failed; the CUDA error was read and cleared        */
  XNOR_ERR_TIMEOUT = 4,     /* a bounded device-side wait gave up (see xnor_check_device)    */
  XNOR_ERR_BOUNDS = 5       /* checking build only: a kernel computed an address outside its
                               buffer; the access was skipped (see xnor_built_with_bounds_check) */
} xnor_status;

/* Geometry of one convolution layer.  Square or rectangular filters, one
 * stride and one zero-padding amount for both axes, no groups, no dilation.
 * `flags` selects two options the paper mentions around the block (Section
 * 3.2, "Training XNOR-Networks"); 0 is the block as Eq. 11 states it, and a
 * descriptor initialised with nine values (C aggregate initialisation) has
 * flags = 0.  Unknown bits give INVALID_ARG. */
typedef struct {
  int N, C_in, H, W;
  int C_out, k_h, k_w;
  int stride, pad;
  int flags;
} xnor_conv_desc;

/* "We can insert a non-binary activation (e.g. ReLU) after binary
 * convolution": the BinConv calls write max(v, 0) instead of v, where v is the
 * value after the K alpha scaling and after the shortcut add, if any (NaN
 * gives 0).  Ignored by the BinActiv calls. */
#define XNOR_FLAG_RELU 1
/* Border variant of K = A * k: the box filter divides by the number of taps
 * that lie inside the image instead of k_h*k_w, so K is the mean of A over the
 * input values the window really sees (0 for a window wholly in the padding).
 * Read by the BinActiv calls (they make K); ignored by the BinConv calls. */
#define XNOR_FLAG_K_VALID_TAPS 2

/* Library version: major*10000 + minor*100 + patch. */
int xnor_version(void);

/* 1 when the library was compiled with -DXNOR_BOUNDS_CHECK, else 0.  In that build the
 * tensor-core BinConv kernel compares every shared-memory address its producers compute and
 * every global index its epilogue stores to with the extent of the buffer, skips an access that
 * fails and records it; xnor_check_device then returns XNOR_ERR_BOUNDS (once).  The ordinary
 * build carries none of these checks.  Meant for running the parity suite once over a change. */
int xnor_built_with_bounds_check(void);

/* Static, human-readable name of a status code. */
const char *xnor_status_string(xnor_status s);

/* ceil(C_in / 32): 32-bit words per packed pixel or filter tap. */
size_t xnor_words_per_pixel(int C_in);

/* Output extent (in + 2*pad - k)/stride + 1, or 0 when the filter does not fit. */
int xnor_out_extent(int in, int k, int stride, int pad);

/*
 * Weight binarisation -- Section 3.1, Eq. 4 and Eq. 6 (the two assignments in
 * the filter loop of Algorithm 1): per filter, B = sign(W) and
 * alpha = ||W||_1 / n with n = C_in*k_h*k_w.  Done once per layer at
 * inference; the real-valued weights are not needed afterwards.
 *
 *   w         in   fp32 [C_out][C_in][k_h][k_w]
 *   w_packed  out  u32  [P][C_out][2], P = ceil(k_h*k_w*Cw / 2): sign bits in
 *                  "word-pair-major" order.  With f = (ky*k_w + kx)*Cw + cw the
 *                  index of a 32-channel word inside a filter, word f of filter
 *                  co is element [f/2][co][f%2]; when k_h*k_w*Cw is odd the last
 *                  pair is padded with a 0 word.  (Words 2j and 2j+1 of all
 *                  filters - one 64-channel step of the contraction - are
 *                  contiguous, which is how the convolution reads them.)
 *   alpha     out  fp32 [C_out]
 *
 * INVALID_ARG: null or misaligned pointer, non-positive size.
 * UNSUPPORTED: k_h*k_w*Cw > 12288 words per filter (does not fit the staging buffer).
 */
xnor_status xnor_binarize_weights(const float *w, int C_out, int C_in, int k_h, int k_w,
                                  uint32_t *w_packed, float *alpha, void *cuda_stream);

/*
 * BatchNorm affine + BinActiv -- Section 3.2, "Binary Convolution" and the
 * B-A-C-P block order of "Training XNOR-Networks": the input is normalised,
 * then BinActiv produces sign(I) and the scaling map K = A * k, where
 * A = (sum over channels of |I|)/c and k is the k_h x k_w filter with all
 * entries 1/(k_h*k_w).
 *
 *   x         in   fp32 [N][C_in][H][W]
 *   bn_scale  in   fp32 [C_in]  or NULL     y = fmaf(bn_scale[c], x, bn_shift[c]),
 *   bn_shift  in   fp32 [C_in]  or NULL     one fused rounding; both NULL = identity
 *   d         in   host pointer; C_out is ignored
 *   x_packed  out  u32  [N][H][W][Cw]       bit = (y >= 0)
 *   A         out  fp32 [N][H][W]           channel mean of |y|; also the scratch the
 *                                           K kernel reads, so it must not be NULL
 *   K         out  fp32 [N][H_out][W_out]   box filter of zero-padded A at the
 *                                           convolution's own output positions, divisor
 *                                           always k_h*k_w (XNOR_FLAG_K_VALID_TAPS:
 *                                           the number of in-image taps)
 *
 * INVALID_ARG: null/misaligned pointer (bn_* may both be NULL, not just one),
 * non-positive size, stride < 1, pad < 0, filter larger than the padded image.
 * UNSUPPORTED (checked before anything is launched): N > 65535; C_in > 2976
 * with a BatchNorm affine or C_in > 8960 without (the packed words of a group
 * of pixels are staged in shared memory).
 */
xnor_status xnor_binactiv(const float *x, const float *bn_scale, const float *bn_shift,
                          const xnor_conv_desc *d, uint32_t *x_packed, float *A, float *K,
                          void *cuda_stream);

/*
 * How many kernels xnor_binactiv launches for this call: 2 (pack + A, then the box
 * filter for K) or 1.  One kernel serves inputs whose planes are not a multiple of
 * four pixels (H*W % 4 != 0, at most 2048 pixels) when C_in % 8 == 0 and N is at least
 * half the SM count: a block then streams whole images and forms K from the A it
 * holds.  Both paths give the same bits; A (and K) may differ in the last place, the
 * channel sums being taken in another order.  0 for a bad descriptor or a shape
 * xnor_binactiv refuses.  has_bn != 0 = with bn_scale / bn_shift.
 */
int xnor_binactiv_launches(const xnor_conv_desc *d, int has_bn);
/* The same for xnor_binactiv_kbit (below): its one-kernel path has the same conditions, with
 * k times the packed words of an image staged in shared memory.  0: bad arguments. */
int xnor_binactiv_kbit_launches(const xnor_conv_desc *d, int kbits, int has_bn);

/*
 * xnor_binactiv without a caller-supplied A buffer.  (The paper has no
 * counterpart; this exists for callers that cannot allocate.)
 *
 * xnor_binactiv needs N*H*W floats of device memory for the A plane, which the
 * box filter reads back to make K.  Some callers have no way to provide it:
 * code that runs where cudaMalloc is not permitted (inside a real-time or
 * pre-planned memory budget, in a plug-in that is handed its input and output
 * buffers and nothing else), or that only needs x_packed and K and has no use
 * for A.  For them this entry point keeps A in a fixed array inside the library:
 * XNOR_BINACTIV_STATIC_MAX_PIXELS floats (4 MiB) of device memory, held by
 * every GPU that has loaded the library until the process exits.  The call
 * allocates nothing and frees nothing, directly or through any other library.
 *
 *   x, bn_scale, bn_shift, d, x_packed, K   exactly as for xnor_binactiv; the
 *                                           results are bit-identical to it
 *
 * UNSUPPORTED: N*H*W > XNOR_BINACTIV_STATIC_MAX_PIXELS (nothing is launched;
 * split the batch or use xnor_binactiv).  INVALID_ARG as for xnor_binactiv.
 *
 * The first call on each device looks up the array's device address (with
 * that device current); make that first call outside any stream capture.
 * All calls on one device share the one array: two calls whose kernels can
 * overlap on the GPU (different streams without an ordering between them)
 * race on it and must be serialised by the caller.  The array keeps whatever
 * the last call left; nothing has to be cleared, because each call writes
 * every element it later reads.
 */
#define XNOR_BINACTIV_STATIC_MAX_PIXELS (1u << 20)
xnor_status xnor_binactiv_static(const float *x, const float *bn_scale, const float *bn_shift,
                                 const xnor_conv_desc *d, uint32_t *x_packed, float *K,
                                 void *cuda_stream);

/*
 * BinConv -- Eq. 11: out = (sign(I) (*) sign(W)) (.) K alpha, where (*) is the
 * convolution evaluated with XNOR and bit-count (Section 3.2).  K is shared
 * by all filters of the layer and differs per image; alpha is per filter.
 *
 *   x_packed  in   u32  [N][H][W][Cw]            from xnor_binactiv
 *   w_packed  in   u32  [P][C_out][2]             from xnor_binarize_weights
 *   alpha     in   fp32 [C_out]
 *   K         in   fp32 [N][H_out][W_out]
 *   residual  in   fp32 [N][C_out][H_out][W_out] or NULL; added after the scaling
 *                  (ResNet shortcut); may be the same buffer as out
 *   out       out  fp32 [N][C_out][H_out][W_out]
 *   acc_out   out  i32  [N][C_out][H_out][W_out] or NULL; the exact integer result of
 *                  sign(I) (*) sign(W) (sum over in-image taps of +-1 products), for
 *                  verification
 *
 * d->flags & XNOR_FLAG_RELU: out = max(., 0) of the above (after the residual add).
 *
 * INVALID_ARG as above.  UNSUPPORTED: k_h or k_w > 11, C_in*k_h*k_w >= 2^24
 * (the integer result must be exact in fp32), or a shape no engine covers
 * (strides above 2 with an input patch larger than the CUDA-core kernel's
 * shared memory).
 */
xnor_status xnor_conv2d_forward(const uint32_t *x_packed, const uint32_t *w_packed,
                                const float *alpha, const float *K, const float *residual,
                                const xnor_conv_desc *d, float *out, int32_t *acc_out,
                                void *cuda_stream);

/*
 * k-bit activations -- Section 3.2, "k-bit Quantization": the block with
 *   q_k(y) = 2([(2^k - 1)(y + 1)/2]/(2^k - 1) - 1/2)
 * in place of sign(y); [.] rounds to the nearest integer, y in [-1, 1].  Everything
 * else of the block (A, K, alpha, Eq. 11's scaling) stays as it is.
 * Readings where the paper is silent: y outside [-1, 1] is clipped; ties round up,
 * which makes k = 1 exactly sign() (+1 at zero); the rounding decision is a
 * comparison in fp32: [.] >= j exactly when y >= fp32((2j - 1)/(2^k - 1) - 1).
 *
 * xnor_binactiv_kbit is xnor_binactiv with
 *   x_planes  out  u32 [kbits][N][H][W][Cw]   plane p holds bit p of the index
 *                  i = [.] in 0 .. 2^k - 1 of every value (the level is
 *                  (2i - (2^k - 1))/(2^k - 1) = sum_p 2^p (2 b_p - 1) / (2^k - 1));
 *                  for kbits = 1 the one plane is xnor_binactiv's x_packed.
 * xnor_conv2d_forward_kbit is xnor_conv2d_forward on those planes:
 *   out = (q_k(I) (*) sign(W)) (.) K alpha (+ residual), one pass of the binary
 *   convolution per plane, each adding D_p K alpha 2^p/(2^k - 1) to the output;
 *   acc_out (nullable) receives the exact integer sum over level codes,
 *   sum_p 2^p D_p = (2^k - 1) (q_k(I) (*) sign(W)).
 * 1 <= kbits <= 7 (INVALID_ARG otherwise); other errors as for the 1-bit calls;
 * for kbits > 1 the convolution needs N*H*W*Cw to be a multiple of 4 (planes
 * stay 16-byte aligned; UNSUPPORTED otherwise) and, with a residual that is not
 * `out` itself, reads it in the first pass only.
 */
xnor_status xnor_binactiv_kbit(const float *x, const float *bn_scale, const float *bn_shift,
                               const xnor_conv_desc *d, int kbits, uint32_t *x_planes, float *A,
                               float *K, void *cuda_stream);
xnor_status xnor_conv2d_forward_kbit(const uint32_t *x_planes, int kbits, const uint32_t *w_packed,
                                     const float *alpha, const float *K, const float *residual,
                                     const xnor_conv_desc *d, float *out, int32_t *acc_out,
                                     void *cuda_stream);

/*
 * Binary-Weight-Network convolution -- Section 3.1, Eq. 1:
 *   I * W ~ (I (+) B) alpha,
 * real-valued inputs, B = sign(W) and alpha from xnor_binarize_weights; (+) is a
 * convolution that only adds and subtracts input values.  The inputs are rounded
 * once to bfloat16 (round to nearest even) and the signed sums run on the tensor
 * cores as bf16 x (+-1) products (exact) accumulated in fp32; then
 *   out = sum * alpha[co] (+ residual), max(., 0) with XNOR_FLAG_RELU.
 * Two calls, like BinActiv + BinConv:
 *   xnor_bwn_prepare_input   x fp32 [N][C_in][H][W] (after the optional BatchNorm
 *       affine y = fmaf(bn_scale[c], x, bn_shift[c])) -> x_stream, the bfloat16 values
 *       in the order the convolution reads them: for each of the stride^2 phases of the
 *       input, the pixels as one stream with zero pixels where the filter overhangs the
 *       image, C_in padded with zeros to a multiple of 16.  xnor_bwn_input_elems(d)
 *       gives the number of 16-bit elements of x_stream for the geometry (0: bad
 *       descriptor); the layout is private to the two calls.
 *   xnor_bwn_conv2d_forward  x_stream, w_packed u32 [P][C_out][2], alpha fp32 [C_out],
 *       residual fp32 [N][C_out][H_out][W_out] or NULL (may be `out`) ->
 *       out fp32 [N][C_out][H_out][W_out].
 * INVALID_ARG as for the other calls.  UNSUPPORTED (nothing launched): stride > 2,
 * more than 121 filter taps, a tile's input window of more than 256 stream positions
 * (roughly (k_h - 1) * (W + k_w) > 120 at stride 1), or a window that does not fit
 * shared memory beside two weight stages (C_in above ~600 at 3x3 on small images).
 * Device-side waits are bounded as in xnor_conv2d_forward (xnor_check_device).
 */
size_t xnor_bwn_input_elems(const xnor_conv_desc *d);
xnor_status xnor_bwn_prepare_input(const float *x, const float *bn_scale, const float *bn_shift,
                                   const xnor_conv_desc *d, uint16_t *x_stream, void *cuda_stream);
xnor_status xnor_bwn_conv2d_forward(const uint16_t *x_stream, const uint32_t *w_packed,
                                    const float *alpha, const float *residual,
                                    const xnor_conv_desc *d, float *out, void *cuda_stream);

/*
 * Backward convolution with a binarised gradient -- Section 3.2, "Binary Gradient":
 * the convolution between the weight filters and the gradient that bounds the
 * backward pass of a layer, with the gradient binarised like the forward operands
 * but scaled by max_i |g_i| (not by the mean of Eq. 6), and, as in Algorithm 1,
 * the binarised filters alpha * sign(W).  For the forward layer described by d
 * (stride 1, k_h = k_w), with g the gradient at the convolution's output,
 *   gmax[n]            = max over image n of |g|
 *   grad_in[n][c][y][x] = sum_{co,ky,kx} alpha[co] sign(W[co][c][ky][kx]) gmax[n]
 *                                        sign(g[n][co][y + pad - ky][x + pad - kx])
 * (taps outside g contribute 0; sign(0) = +1): the gradient with respect to the
 * convolution's input.  alpha sits inside the sum over the filters, so this is a
 * convolution of the real tensor gmax alpha[co] sign(g) with +-1 filters: it runs
 * on the Binary-Weight kernel (above), each product gmax[n] * alpha[co] formed in
 * fp32 and rounded once to bfloat16, sums in fp32.
 *   xnor_binarize_weights_transposed   w fp32 [C_out][C_in][k_h][k_w] ->
 *       wT_packed u32 [P'][C_in][2], P' = ceil(k_h*k_w*ceil(C_out/32) / 2): the sign
 *       bits as the backward convolution contracts them (channels = the filters co,
 *       taps turned by 180 degrees), word-pair-major like w_packed.  Once per layer.
 *   xnor_binary_gradient_backward   g fp32 [N][C_out][H_out][W_out], wT_packed,
 *       alpha fp32 [C_out] (from xnor_binarize_weights) -> gmax fp32 [N],
 *       grad_in fp32 [N][C_in][H][W]; g_stream is scratch of
 *       xnor_bgrad_stream_elems(d) 16-bit elements (0: bad descriptor or unsupported).
 * INVALID_ARG as for the other calls.  UNSUPPORTED (nothing launched): stride != 1,
 * k_h != k_w, N > 65535, or a geometry the Binary-Weight kernel refuses (its limits
 * apply to the convolution of [C_out][H_out][W_out] with pad k - 1 - pad).
 */
size_t xnor_bgrad_stream_elems(const xnor_conv_desc *d);
xnor_status xnor_binarize_weights_transposed(const float *w, int C_out, int C_in, int k_h, int k_w,
                                             uint32_t *wT_packed, void *cuda_stream);
xnor_status xnor_binary_gradient_backward(const float *g, const uint32_t *wT_packed,
                                          const float *alpha, const xnor_conv_desc *d, float *gmax,
                                          uint16_t *g_stream, float *grad_in, void *cuda_stream);

/*
 * Full-precision 1x1 strided convolution without bias: the projection
 * shortcut ("type B") of the ResNet-18 variant the paper binarises
 * (Section 4.2).  Its result is the `residual` of a block's second BinConv.
 *
 *   x    in   fp32 [N][C_in][H][W]
 *   w    in   fp32 [C_out][C_in]
 *   out  out  fp32 [N][C_out][(H-1)/stride+1][(W-1)/stride+1]
 */
xnor_status xnor_shortcut_conv1x1(const float *x, const float *w, int N, int C_in, int H, int W,
                                  int C_out, int stride, float *out, void *cuda_stream);

/*
 * BinConv with the NEXT layer's BinActiv fused into its epilogue.  The block
 * order of Section 3.2 makes the output of one BinConv (after the residual add,
 * where there is one) the input of the next BatchNorm + BinActiv; the epilogue
 * holds those fp32 values in registers, so it can emit what the next BinConv
 * consumes without the fp32 tensor making a round trip through memory:
 *   y = fmaf(next_scale[co], out[n][co][p], next_shift[co])   (identity if both NULL)
 *   x_packed_next  u32 [N][H_out][W_out][ceil(C_out/32)]   bit = (y >= 0), along the filters
 *   A_parts        fp32 [parts][N][H_out][W_out]           partial sums over filters of |y|
 * `out` may be NULL (the fp32 tensor is then not written at all) or a buffer as
 * in xnor_conv2d_forward; residual as there; no acc_out.  Values of out, and
 * therefore the sign bits, are the ones xnor_conv2d_forward produces.
 * xnor_conv2d_binactiv_parts(d) gives `parts` for the shape and the engine in
 * force (set the engine before asking, do not change it in between); 0 means
 * the fused kernel does not cover the shape (needs the tensor-core engine and
 * C_out % 32 == 0): the call then returns UNSUPPORTED and the caller runs
 * xnor_conv2d_forward + xnor_binactiv instead.
 * xnor_binactiv_finish completes the next layer's BinActiv: A = (sum of the
 * parts, in index order) / C_in of d_next, K = box filter of A for d_next's
 * geometry (d_next: N, C_in = this C_out, H = H_out, W = W_out, its own k, stride, pad).
 */
int xnor_conv2d_binactiv_parts(const xnor_conv_desc *d);
xnor_status xnor_conv2d_forward_binactiv(const uint32_t *x_packed, const uint32_t *w_packed,
                                         const float *alpha, const float *K, const float *residual,
                                         const xnor_conv_desc *d, float *out, const float *next_scale,
                                         const float *next_shift, uint32_t *x_packed_next,
                                         float *A_parts, void *cuda_stream);
xnor_status xnor_binactiv_finish(const float *A_parts, int parts, const xnor_conv_desc *d_next,
                                 float *A, float *K, void *cuda_stream);

/*
 * The Pool layer that closes the block (Section 3.2, "Training XNOR-Networks":
 * the order is BatchNorm, BinActiv, BinConv, Pool, with an optional ReLU after
 * the binary convolution): max pooling of BinConv's output.
 *   x     in   fp32  [N][C][H][W]           device, 16-byte aligned
 *   out   out  fp32  [N][C][H_out][W_out]   H_out = (H + 2 pad - k) / stride + 1 rounded down
 *   relu  != 0: max(v, 0) is applied to every input value first
 * A tap outside the image takes no part in the maximum (0 <= pad < k, so every
 * window holds at least one pixel).  Maxima of fp32 values are exact: results
 * are bit-identical to the plain definition.  Asynchronous on `cuda_stream`.
 * INVALID_ARG for null/misaligned pointers, non-positive sizes, pad outside
 * [0, k), k larger than the padded image; UNSUPPORTED for k > 11.
 */
xnor_status xnor_maxpool2d(const float *x, int N, int C, int H, int W, int k, int stride, int pad,
                           int relu, float *out, void *cuda_stream);

/*
 * Which BinConv engine xnor_conv2d_forward uses.  XNOR_ENGINE_AUTO (default)
 * picks by shape: the tensor-core engine where it applies, else the CUDA-core
 * one.  Meant for tests and measurements.  This is the library's only
 * process-wide setting: an atomic that every BinConv call reads once at its
 * start, so a call uses one engine throughout and a change made by another
 * thread applies to the calls that start after it; a program that wants
 * different engines in different threads must order those calls itself.
 * With an engine forced, xnor_conv2d_forward returns UNSUPPORTED for shapes
 * that engine does not cover.
 *   XNOR_ENGINE_POPC   CUDA-core XOR + population count, any supported shape
 *   XNOR_ENGINE_UMMA   5th-generation tensor cores (tcgen05), 4-bit (e2m1)
 *                      operands built from the sign bits, exact fp32
 *                      accumulation of integers; strides 1 and 2, shapes whose
 *                      activation patch fits shared memory.  The expanded
 *                      filters of a slab stay in shared memory while a CTA
 *                      walks the pixel tiles, when they fit; CTA pairs (one
 *                      MMA instruction drives two SMs, each CTA holding half
 *                      of the slab's filters) where the shape allows
 *   The remaining values pin one variant of that engine (for tests and
 *   measurements):
 *   XNOR_ENGINE_UMMA_STREAM       one CTA per SM, filters re-expanded through
 *                                 a ring of stages for every work item
 *   XNOR_ENGINE_UMMA_SINGLE       one CTA per SM, resident filters if they fit
 *   XNOR_ENGINE_UMMA_PAIR         CTA pairs, resident filters if they fit
 *   XNOR_ENGINE_UMMA_PAIR_STREAM  CTA pairs, filters always re-expanded
 */
typedef enum {
  XNOR_ENGINE_AUTO = 0,
  XNOR_ENGINE_POPC = 1,
  XNOR_ENGINE_UMMA = 2,
  XNOR_ENGINE_UMMA_STREAM = 3,
  XNOR_ENGINE_UMMA_SINGLE = 4,
  XNOR_ENGINE_UMMA_PAIR = 5,
  XNOR_ENGINE_UMMA_PAIR_STREAM = 6
} xnor_engine;
xnor_status xnor_set_engine(xnor_engine e);
xnor_engine xnor_get_engine(void);

/*
 * Measures, on the current device, the per-clock rates of the two pipes a binary
 * convolution can run on (Section 4.1 reasons in binary operations per clock):
 *   mma_mac_per_clk_per_sm   1-bit multiply-accumulates per SM clock of the tensor
 *                            cores on the instruction the BinConv kernel issues
 *                            (tcgen05.mma kind::mxf4 on operands in shared memory,
 *                            128 x 256 x 64 per instruction);
 *   popc_per_clk_per_sm      32-bit population counts (with their XOR and add) per
 *                            SM clock on the CUDA cores (one covers 32 1-bit MACs).
 * Both are HOST pointers.  Multiply by the number of SMs and the SM clock observed
 * while the kernels of interest run to get a peak in operations per second.  The
 * call launches two short kernels (about a millisecond each, twice) on `cuda_stream`
 * and SYNCHRONISES that stream; it allocates nothing.  For benchmarks, not for the
 * data path.  XNOR_ERR_CUDA when a launch fails or a bounded wait inside gives up.
 */
xnor_status xnor_measure_peaks(double *mma_mac_per_clk_per_sm, double *popc_per_clk_per_sm,
                               void *cuda_stream);

/*
 * The one call that synchronises: waits for `cuda_stream`, then reads the
 * device-side status word.  Every wait inside the tensor-core kernel (on a
 * shared-memory barrier) is bounded; a wait that expires records
 * XNOR_ERR_TIMEOUT there, the kernel stops issuing work, releases its tensor
 * memory and returns, and the outputs of that launch are undefined.  Returns
 * XNOR_OK, XNOR_ERR_TIMEOUT (the word is then cleared), XNOR_ERR_CUDA or, from a
 * checking build, XNOR_ERR_BOUNDS.
 */
xnor_status xnor_check_device(void *cuda_stream);

/*
 * Exercises that error path without touching any data: launches on
 * `cuda_stream` one warp that waits, with a limit of about a millisecond, on
 * a barrier that nothing signals.  The wait gives up by itself, so the next
 * xnor_check_device returns XNOR_ERR_TIMEOUT once and the device stays
 * usable.  No counterpart in the paper; meant for tests of the bounded waits.
 * Returns XNOR_OK or XNOR_ERR_CUDA (launch failure).
 */
xnor_status xnor_selftest_wait_timeout(void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* XNOR_H_ */
