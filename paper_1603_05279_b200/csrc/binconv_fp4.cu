// BinConv on the 5th-generation tensor cores with 4-bit operands (Eq. 11).
//
// sign(I) (*) sign(W) is an exact integer contraction.  It runs here as an
// implicit GEMM on tcgen05.mma kind::mxf4 (e2m1 operands, unit block scales,
// fp32 accumulation in tensor memory, exact because every partial sum is an
// integer below 2^24).  HBM only ever sees the 1-bit packed words; each CTA
// expands what it needs into shared memory.
//
//  GEMM roles.  D[filter][pixel] = sum_k Wt[filter][k] * X[pixel][k]:
//    A (M = 128 rows)  = a 128-filter slab of weights, streamed through a ring
//                        of shared-memory stages (one (tap, 64 or 128 channels)
//                        piece per stage) that the producer warps expand from bits;
//    B (N <= 224 rows) = activations.  All images form one long virtual stream
//                        of pixels: every image row is preceded by `pad` zero
//                        pixels and every image by `pad` zero rows (row width
//                        Wp = W + pad, image height Hp = H + pad; the zeros right
//                        of a row / below an image are the ones that precede the
//                        next row / image).  With GEMM column n = stream index of
//                        the output pixel, filter tap (ky,kx) reads stream pixel
//                        n + ky*Wp + kx: a pure shift.  A CTA owns NP consecutive
//                        stream positions and expands the NP + (kh-1)*Wp + (kw-1)
//                        pixels they touch ONCE; every tap's B operand is that
//                        same patch at a shifted start address (no-swizzle K-major
//                        layout: 8 pixels x 16 bytes per core matrix, pixels
//                        contiguous).  Zero pixels and the channel tail expand to
//                        0, so padded taps contribute exactly 0 with no mask.
//                        Stream positions that are padding yield junk columns that
//                        are never stored.
//
//  Operand encodings.  A packed word holds 32 sign bits; it becomes 32 e2m1
//  nibbles in four registers, register r holding channels r, r+4, ..., r+28.
//  Weights need ONE logic op per register: a single set bit inside a nibble is
//  already a valid e2m1 number (0x1 = 0.5, 0x2 = 1, 0x4 = 2), so with
//  beta = sign bit, value = beta * {0.5, 1, 2, 2} for r = 0..3.  Activations
//  carry the reciprocal magnitude and the sign, a * {2, 1, 0.5, 0.5} with
//  a = +-1 (0 for padding / channel tail).  Every product is a * beta, so
//  D = sum(a * beta), and with sign(W) = 2 beta - 1
//      sum(a * sign(W)) = 2 D - S,   S = sum of a over the window,
//  where S is a box sum of per-pixel values (2 popcount - channels) that the
//  activation expansion leaves in shared memory.
//
//  Warp 0 issues the MMAs; warps 1..8 expand operands and then run the
//  epilogue: accumulators go TMEM -> registers -> shared memory (transposed)
//  -> coalesced NCHW stores of (2D - S) * K * alpha (+ residual).
//  Every wait is bounded: on expiry the CTA records XNOR_ERR_TIMEOUT in a
//  device status word, stops issuing work, frees its tensor memory and exits.
#include "common.cuh"
#include "umma_common.cuh"

namespace xnor {

__device__ int g_status_fp4 = 0;
#ifdef XNOR_TRACE
__device__ long long g_trace[256];
#define TRACE(i) do { if (blockIdx.x == gridDim.x / 2 && blockIdx.y == 0) g_trace[i] = clock64(); } while (0)
#else
#define TRACE(i) do {} while (0)
#endif

namespace {

using namespace umma;

constexpr int kProducerWarps = 8;
constexpr int kProducers = 32 * kProducerWarps;
constexpr int kThreads = 32 + kProducers;
constexpr int kFilters = 128;        // M: filters per CTA = tensor-memory lanes
constexpr int kMaxPix = 224;         // N: stream pixels per CTA = accumulator columns
constexpr int kSfCols = 32;          // tensor-memory columns holding the unit block scales
constexpr int kTmemCols = 256;       // accumulator + scales, power of two; two CTAs per SM
constexpr int kMaxStages = 8;
constexpr int kPrefetch = 4;         // weight stages whose packed words are in flight
constexpr int kMaxChunkWords = 16;   // channel words of the patch resident at a time
constexpr size_t kCtrlBytes = 256;
constexpr size_t kSmemBudget = 115000;   // planning budget: two CTAs per SM
constexpr size_t kSmemCap = 115712;      // (228 KB per SM) / 2 - 1 KB reserved per CTA

struct Fp4Params {
  const uint32_t *xp, *wp;
  const float *alpha, *K, *residual;
  float *out;
  int32_t *acc_out;
  int N, C, H, W, Co, kh, kw, pad, Ho, Wo, Cw, Hp, Wp;
  long long L;         // stream length N*Hp*Wp
  int NP;              // stream positions per CTA, multiple of 32, <= kMaxPix
  int ppix;            // stream pixels staged per CTA (NP + halo, rounded up to 8)
  int cwc;             // channel words per patch chunk (even unless it is all of Cw)
  int stages;
  uint32_t region0;    // bytes shared by {patch + weight stages} and the epilogue's transpose tile
  uint32_t idesc;
  uint32_t tail_mask;  // bits of real channels in the last word (all ones if C % 32 == 0)
};

__device__ __forceinline__ void umma_mxf4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t sfa, uint32_t sfb,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
      : "memory");
}

// beta * {0.5, 1, 2, 2}: one set bit per nibble
__device__ __forceinline__ void expand_weights(uint32_t w, uint32_t v[4]) {
  v[0] = w & 0x11111111u;
  v[1] = w & 0x22222222u;
  v[2] = w & 0x44444444u;
  v[3] = (w >> 1) & 0x44444444u;
}

// a * {2, 1, 0.5, 0.5}: e2m1 codes 0x4/0xC, 0x2/0xA, 0x1/0x9 (sign is bit 3)
__device__ __forceinline__ void expand_activations(uint32_t w, uint32_t v[4]) {
  v[0] = 0xCCCCCCCCu - ((w & 0x11111111u) << 3);
  v[1] = 0xAAAAAAAAu - (((w >> 1) & 0x11111111u) << 3);
  v[2] = 0x99999999u - (((w >> 2) & 0x11111111u) << 3);
  v[3] = 0x99999999u - (((w >> 3) & 0x11111111u) << 3);
}

__device__ __forceinline__ void bar_sync_producers() {
  asm volatile("bar.sync 1, %0;" ::"n"(kProducers) : "memory");
}

// WPS: channel words per weight stage (2 or 4; one MMA consumes two).
template <int WPS>
__global__ void __launch_bounds__(kThreads, 2) binconv_fp4_kernel(const Fp4Params P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int taps = P.kh * P.kw;
  const int NP = P.NP;
  const int cwc_e = (P.cwc + 1) & ~1;                         // patch planes (even)
  const uint32_t a_lbo = (uint32_t)P.ppix * 16u;              // patch plane = one channel word
  constexpr uint32_t w_lbo = (uint32_t)kFilters * 16u;        // weight-stage plane
  constexpr uint32_t stage_bytes = (uint32_t)WPS * w_lbo;
  const uint32_t patch_bytes = (uint32_t)cwc_e * a_lbo;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t patch_addr = smem_base;
  const uint32_t stage_addr = patch_addr + patch_bytes;
  uint8_t *ctrl = smem + P.region0;
  uint64_t *bars = reinterpret_cast<uint64_t *>(ctrl);
  // bars: [0,S) full, [S,2S) empty, 2S patch_full, 2S+1 patch_free, 2S+2 accum_full
  const uint32_t bar0 = smem_u32(bars);
  const int S = P.stages;
  const uint32_t patch_full = bar0 + 8u * (2 * S), patch_free = patch_full + 8u,
                 accum_full = patch_full + 16u;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kMaxStages + 4);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  int *pix_sum = reinterpret_cast<int *>(ctrl + kCtrlBytes);     // [ppix] sum over channels of a
  float *alpha_sm = reinterpret_cast<float *>(pix_sum + P.ppix); // [kFilters]
  float *k_sm = alpha_sm + kFilters;                             // [NP] K of the output pixel
  int *img_sm = reinterpret_cast<int *>(k_sm + NP);              // [NP] image index, -1 = no output
  int *pix_sm = img_sm + NP;                                     // [NP] oy*Wo + ox
  int *win_sm = pix_sm + NP;                                     // [NP] S: window sum of a

  if (tid == 0) TRACE(0);
  for (int q = tid; q < P.ppix; q += kThreads) pix_sum[q] = 0;
  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < S; ++s) {
        mbar_init(bar0 + 8u * s, kProducerWarps);
        mbar_init(bar0 + 8u * (S + s), 1);
      }
      mbar_init(patch_full, kProducerWarps);
      mbar_init(patch_free, 1);
      mbar_init(accum_full, 1);
      *abort_flag = 0;
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_sf = tmem_base + (uint32_t)kMaxPix;   // columns [224, 256)
  if (tid == 0) TRACE(1);

  const uint32_t m0 = blockIdx.x * (uint32_t)NP;
  const int co0 = blockIdx.y * kFilters;
  const int nchunks = (P.Cw + P.cwc - 1) / P.cwc;

  if (warp == 0) {
    // ------------------------------------------------------------ MMA issuer
    uint32_t accumulate = 0, ph = 0;
    int s = 0;
    bool ok = true;
    for (int cc = 0; cc < nchunks && ok; ++cc) {
      const int cwn = min(P.cwc, P.Cw - cc * P.cwc);
      const int cwn_e = (cwn + 1) & ~1;
      ok = mbar_wait(patch_full, cc & 1, abort_flag, &g_status_fp4);
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) TRACE(2);
      int kx = 0;
      uint32_t b_tap = patch_addr;                       // + (ky*Wp + kx) * 16
      for (int tap = 0; tap < taps && ok; ++tap) {
        for (int wb = 0; wb < cwn_e; wb += WPS) {
          ok = mbar_wait(bar0 + 8u * s, ph, abort_flag, &g_status_fp4);
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
            uint32_t b_addr = b_tap + (uint32_t)wb * a_lbo;
            uint32_t a_addr = stage_addr + s * stage_bytes;
#pragma unroll
            for (int wi = 0; wi < WPS; wi += 2) {
              if (wi == 0 || wb + wi < cwn_e) {
                umma_mxf4(tmem_base, make_desc(a_addr, w_lbo, 128u), make_desc(b_addr, a_lbo, 128u),
                          P.idesc, tmem_sf, tmem_sf, accumulate);
                accumulate = 1;
                a_addr += 2u * w_lbo;
                b_addr += 2u * a_lbo;
              }
            }
            umma_commit(bar0 + 8u * (S + s));
          }
          __syncwarp();
          if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (++kx == P.kw) { kx = 0; b_tap += (uint32_t)(P.Wp - P.kw + 1) * 16u; }
        else b_tap += 16u;
      }
      if (ok && lane == 0) umma_commit(patch_free);
      __syncwarp();
    }
    if (ok && lane == 0) umma_commit(accum_full);
    if (lane == 0) TRACE(3);
    __syncwarp();
  } else {
    // ------------------------------------------------------------ producers
    const int pt = tid - 32;
    uint32_t ph = 1;          // parity to wait for on the empty barriers
    int s = 0;
    bool ok = true;
    const int crem = P.C - 32 * (P.Cw - 1);
    const size_t HoWo = (size_t)P.Ho * P.Wo;

    // unit block scales (ue8m0 1.0 = 0x7F) in every lane of the scale columns
    if (warp <= 4) {
      const uint32_t taddr = tmem_sf + ((uint32_t)((warp & 3) * 32) << 16);
      const uint32_t one = 0x7F7F7F7Fu;
#pragma unroll
      for (int k = 0; k < kSfCols / 8; ++k)
        asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};"
                     ::"r"(taddr + 8u * k), "r"(one) : "memory");
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      tc_fence_before();
    }
    // per-column metadata of the output pixels, and alpha of this filter slab
    if (pt < kFilters) alpha_sm[pt] = co0 + pt < P.Co ? __ldg(P.alpha + co0 + pt) : 0.0f;
    if (pt < NP) {
      const uint32_t m = m0 + (uint32_t)pt;
      int img = -1, pix = 0;
      float kv = 0.0f;
      if (m < (uint32_t)P.L) {
        const uint32_t r = m / (uint32_t)P.Wp;
        const int ox = (int)(m - r * (uint32_t)P.Wp);
        const uint32_t n = r / (uint32_t)P.Hp;
        const int oy = (int)(r - n * (uint32_t)P.Hp);
        if (ox < P.Wo && oy < P.Ho) {
          img = (int)n;
          pix = oy * P.Wo + ox;
          kv = __ldg(P.K + (size_t)n * HoWo + pix);
        }
      }
      img_sm[pt] = img;
      pix_sm[pt] = pix;
      k_sm[pt] = kv;
    }

    for (int cc = 0; cc < nchunks && ok; ++cc) {
      const int cw0 = cc * P.cwc;
      const int cwn = min(P.cwc, P.Cw - cw0);
      const int cwn_e = (cwn + 1) & ~1;
      if (cc > 0) {
        ok = mbar_wait(patch_free, (cc - 1) & 1, abort_flag, &g_status_fp4);
        if (!ok) break;
      }
      // expand the activation patch: one thread per stream pixel, all channel words of
      // the chunk; every global load is issued before the first expansion
      for (int q = pt; q < P.ppix; q += kProducers) {
        const uint32_t sq = m0 + (uint32_t)q;
        const uint32_t *src = nullptr;
        if (sq < (uint32_t)P.L) {
          const uint32_t r = sq / (uint32_t)P.Wp;
          const int c = (int)(sq - r * (uint32_t)P.Wp);
          const uint32_t n = r / (uint32_t)P.Hp;
          const int ry = (int)(r - n * (uint32_t)P.Hp);
          if (c >= P.pad && ry >= P.pad)
            src = P.xp + (((size_t)n * P.H + (ry - P.pad)) * P.W + (c - P.pad)) * P.Cw + cw0;
        }
        uint32_t pw[kMaxChunkWords];
#pragma unroll
        for (int wl = 0; wl < kMaxChunkWords; ++wl)
          pw[wl] = (src != nullptr && wl < cwn) ? __ldg(src + wl) : 0u;
        int psum = 0;
        uint32_t a = patch_addr + (uint32_t)q * 16u;
#pragma unroll
        for (int wl = 0; wl < kMaxChunkWords; ++wl) {
          if (wl < cwn_e) {
            uint32_t v[4] = {0u, 0u, 0u, 0u};
            if (src != nullptr && wl < cwn) {
              expand_activations(pw[wl], v);
              int nreal = 32;
              if (cw0 + wl == P.Cw - 1 && crem != 32) {
                nreal = crem;
#pragma unroll
                for (int r = 0; r < 4; ++r) v[r] &= ((P.tail_mask >> r) & 0x11111111u) * 0xFu;
              }
              psum += 2 * __popc(pw[wl]) - nreal;
            }
            sts128(a, v[0], v[1], v[2], v[3]);
            a += a_lbo;
          }
        }
        pix_sum[q] += psum;
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(patch_full);
      if (pt == 0) TRACE(8);

      // weight stages of this chunk in the issuer's order (tap outer, words inner).
      // Thread = (filter row, parity): it expands the words of its parity in each
      // stage.  kPrefetch register sets hold the packed words of the next stages; a
      // set is refilled right after it is expanded.
      constexpr int WPT = WPS / 2;                    // words per thread per stage
      const int row = pt & (kFilters - 1), par = pt >> 7;
      const int co = co0 + row;
      const bool row_live = co < P.Co;
      const int f_co = row_live ? co : 0;
      int f_word = cw0 + par;                         // word index of (tap f_tap, word f_wb) in the row
      int f_wb = 0, f_tap = row_live ? 0 : taps;      // dead rows never fetch
      uint32_t pf[kPrefetch][WPT];
      auto fetch = [&](uint32_t dst[WPT]) {
        if (f_tap < taps) {
#pragma unroll
          for (int i = 0; i < WPT; ++i)
            dst[i] = f_wb + 2 * i + par < cwn
                         ? __ldg(P.wp + packed_weight_index(P.Co, f_co, f_word + f_wb + 2 * i)) : 0u;
          f_wb += WPS;
          if (f_wb >= cwn_e) { f_wb = 0; ++f_tap; f_word += P.Cw; }
        } else {
#pragma unroll
          for (int i = 0; i < WPT; ++i) dst[i] = 0u;
        }
      };
#pragma unroll
      for (int d = 0; d < kPrefetch; ++d) fetch(pf[d]);
      const uint32_t row_addr = stage_addr + (uint32_t)par * w_lbo + (uint32_t)row * 16u;
      int tap = 0, wb = 0;
      while (tap < taps && ok) {
#pragma unroll
        for (int d = 0; d < kPrefetch; ++d) {
          if (tap < taps && ok) {
            ok = mbar_wait(bar0 + 8u * (S + s), ph, abort_flag, &g_status_fp4);
            if (ok) {
              const uint32_t a = row_addr + s * stage_bytes;
#pragma unroll
              for (int i = 0; i < WPT; ++i) {
                if (i == 0 || wb + 2 * i < cwn_e) {
                  uint32_t v[4];
                  expand_weights(pf[d][i], v);         // 0 for rows beyond C_out
                  sts128(a + (uint32_t)(2 * i) * w_lbo, v[0], v[1], v[2], v[3]);
                }
              }
              fence_proxy_async();
              __syncwarp();
              if (lane == 0) mbar_arrive(bar0 + 8u * s);
              if (++s == S) { s = 0; ph ^= 1u; }
              wb += WPS;
              if (wb >= cwn_e) { wb = 0; ++tap; }
              fetch(pf[d]);
            }
          }
        }
      }
    }
    if (pt == 0) TRACE(9);
    // ------------------------------------------------------------ epilogue
    if (ok) ok = mbar_wait(accum_full, 0, abort_flag, &g_status_fp4);
    if (pt == 0) TRACE(10);
    // window sums S (pix_sum is complete: every chunk was expanded before accum_full)
    if (pt < NP) {
      int wsum = 0;
      if (img_sm[pt] >= 0)
        for (int ky = 0; ky < P.kh; ++ky)
          for (int kx = 0; kx < P.kw; ++kx) wsum += pix_sum[pt + ky * P.Wp + kx];
      win_sm[pt] = wsum;
    }
    tc_fence_after();
    // Accumulators leave tensor memory as [filter lane][pixel column]; NCHW wants lanes
    // along pixels, so each half of the columns is transposed through shared memory
    // (the patch and weight stages are dead by now and are reused as the tile).
    const int NPH = NP / 2;                       // columns per pass, multiple of 16
    const int TS = NPH + 4;                       // tile row stride in words: conflict-free both ways
    int *tile = reinterpret_cast<int *>(smem);
    const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
    const int sub = (warp - 1) >> 2;              // which half of the column blocks
    const int nblk = NPH / 16;
    const int b_begin = sub == 0 ? 0 : (nblk + 1) / 2;
    const int b_end = sub == 0 ? (nblk + 1) / 2 : nblk;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int f0 = (warp - 1) * (kFilters / kProducerWarps);   // 16 filters per warp in pass 2
    const bool plain = P.residual == nullptr && P.acc_out == nullptr;
    for (int h = 0; h < 2; ++h) {
      bar_sync_producers();                       // tile free (and win_sm visible)
      if (ok) {
        int *trow = tile + (quarter * 32 + lane) * TS;
        for (int b = b_begin; b < b_end; ++b) {
          int32_t r[16];
          tmem_ld16(t_lane + (uint32_t)(h * NPH + b * 16), r);
          tmem_wait16(r);
#pragma unroll
          for (int j = 0; j < 16; j += 4) {
            int4 v;
            v.x = __float2int_rn(__int_as_float(r[j]));
            v.y = __float2int_rn(__int_as_float(r[j + 1]));
            v.z = __float2int_rn(__int_as_float(r[j + 2]));
            v.w = __float2int_rn(__int_as_float(r[j + 3]));
            *reinterpret_cast<int4 *>(trow + b * 16 + j) = v;
          }
        }
      }
      bar_sync_producers();                       // tile complete
      if (ok) {
        float al[kFilters / kProducerWarps];
#pragma unroll
        for (int i = 0; i < kFilters / kProducerWarps; ++i) al[i] = alpha_sm[f0 + i];
        const int nf = min(kFilters / kProducerWarps, P.Co - co0 - f0);   // live filters of this warp
        for (int pl = lane; pl < NPH; pl += 32) {
          const int p = h * NPH + pl;
          const int img = img_sm[p];
          if (img < 0) continue;
          const float kv = k_sm[p];
          const int wsum = win_sm[p];
          const size_t o0 = ((size_t)img * P.Co + co0 + f0) * HoWo + pix_sm[p];
          const int *tcol = tile + f0 * TS + pl;
          if (plain && nf == kFilters / kProducerWarps) {
            float *op = P.out + o0;
#pragma unroll
            for (int i = 0; i < kFilters / kProducerWarps; ++i) {
              const int acc = 2 * tcol[i * TS] - wsum;
              *op = __fmul_rn(__fmul_rn((float)acc, kv), al[i]);
              op += HoWo;
            }
          } else {
#pragma unroll
            for (int i = 0; i < kFilters / kProducerWarps; ++i) {
              if (i < nf) {
                const int acc = 2 * tcol[i * TS] - wsum;
                const size_t o = o0 + (size_t)i * HoWo;
                float v = __fmul_rn(__fmul_rn((float)acc, kv), al[i]);
                if (P.residual) v += P.residual[o];
                P.out[o] = v;
                if (P.acc_out) P.acc_out[o] = acc;
              }
            }
          }
        }
      }
    }
    if (pt == 0) TRACE(11);
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0) TRACE(4);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
  }
}

struct Plan {
  int NP, ppix, cwc, wps, stages, mtiles, ftiles;
  uint32_t region0;
  size_t smem;
  bool ok;
};

Plan make_plan(const ConvGeom &g, int sm_count) {
  Plan p{};
  p.ok = false;
  if (g.stride != 1) return p;
  const int Wp = g.W + g.pad, Hp = g.H + g.pad;
  const long long L = (long long)g.N * Hp * Wp;
  if (L >= (1ll << 31) - 2 * kMaxPix) return p;
  const int halo = (g.kh - 1) * Wp + g.kw - 1;
  p.ftiles = (g.Co + kFilters - 1) / kFilters;
  // pixels per CTA: the multiple of 32 (<= 224) that leaves the least idle CTA slots in
  // the last wave of 2 CTAs per SM; ties go to the larger tile
  int best_np = 0;
  double best_cost = 0.0;
  const long long slots = 2ll * (sm_count > 0 ? sm_count : 148);
  for (int np = kMaxPix; np >= 96; np -= 32) {
    const long long ctas = ((L + np - 1) / np) * p.ftiles;
    const long long waves = (ctas + slots - 1) / slots;
    // time ~ waves * (tile work + fixed per-CTA cost expressed in pixels)
    const double cost = (double)waves * (np + 48.0);
    if (best_np == 0 || cost < best_cost * 0.999) { best_np = np; best_cost = cost; }
  }
  p.NP = best_np;
  p.mtiles = (int)((L + p.NP - 1) / p.NP);
  p.ppix = (p.NP + halo + 7) / 8 * 8;
  if ((size_t)p.ppix * 16 >= (1u << 18)) return p;
  const size_t tile_bytes = (size_t)kFilters * (p.NP / 2 + 4) * sizeof(int);
  const size_t fixed = kCtrlBytes + (size_t)p.ppix * sizeof(int) + kFilters * sizeof(float) +
                       (size_t)p.NP * 4 * sizeof(int);
  const size_t plane = (size_t)p.ppix * 16;              // patch bytes per channel word
  const int cw_e = (g.Cw + 1) & ~1;
  // whole channel range resident if it fits with at least 3 stages
  p.cwc = 0;
  for (int wps = 4; wps >= 2; wps -= 2) {
    if (wps == 4 && cw_e % 4 != 0) continue;
    if (g.Cw > kMaxChunkWords) break;
    const size_t stage = (size_t)wps * kFilters * 16;
    if (fixed + plane * cw_e + 3 * stage > kSmemBudget) continue;
    int stages = (int)((kSmemBudget - fixed - plane * cw_e) / stage);
    if (stages > kMaxStages) stages = kMaxStages;
    p.cwc = g.Cw; p.wps = wps; p.stages = stages;
    break;
  }
  if (p.cwc == 0) {   // chunk the channels: 4 stages of 4 words, the rest for the patch
    p.wps = 4; p.stages = 4;
    const size_t stage = (size_t)p.wps * kFilters * 16;
    if (fixed + 4 * stage + 4 * plane > kSmemBudget) return p;
    size_t cwc = (kSmemBudget - fixed - 4 * stage) / plane;
    if (cwc > (size_t)kMaxChunkWords) cwc = kMaxChunkWords;
    cwc &= ~(size_t)3;                                     // chunks start on a stage boundary
    if (cwc > (size_t)g.Cw) cwc = g.Cw;
    p.cwc = (int)cwc;
    if (p.cwc < g.Cw && p.cwc % 4 != 0) return p;
  }
  const size_t work = plane * ((p.cwc + 1) & ~1) + (size_t)p.stages * p.wps * kFilters * 16;
  p.region0 = (uint32_t)((work > tile_bytes ? work : tile_bytes) + 255) / 256 * 256;
  p.smem = p.region0 + fixed;
  if (p.smem > kSmemCap) return p;
  p.ok = true;
  return p;
}

int sm_count_cached() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      (void)cudaGetLastError();
      n = 148;
    }
  }
  return n;
}

}  // namespace

bool umma_fp4_supported(const ConvGeom &g) { return make_plan(g, 148).ok; }

cudaError_t launch_binconv_fp4(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                               const float *K, const float *residual, const ConvGeom &g,
                               float *out, int32_t *acc_out, cudaStream_t st) {
  const Plan pl = make_plan(g, sm_count_cached());
  if (!pl.ok) return cudaErrorInvalidValue;
  Fp4Params P;
  P.xp = xp; P.wp = wp; P.alpha = alpha; P.K = K; P.residual = residual;
  P.out = out; P.acc_out = acc_out;
  P.N = g.N; P.C = g.C; P.H = g.H; P.W = g.W; P.Co = g.Co; P.kh = g.kh; P.kw = g.kw;
  P.pad = g.pad; P.Ho = g.Ho; P.Wo = g.Wo; P.Cw = g.Cw;
  P.Hp = g.H + g.pad; P.Wp = g.W + g.pad;
  P.L = (long long)g.N * P.Hp * P.Wp;
  P.NP = pl.NP; P.ppix = pl.ppix; P.cwc = pl.cwc; P.stages = pl.stages; P.region0 = pl.region0;
  // block-scaled descriptor: e2m1 x e2m1, ue8m0 scales, N = NP, M = 128
  P.idesc = (1u << 7) | (1u << 10) | ((uint32_t)(P.NP >> 3) << 17) | (1u << 23) |
            ((uint32_t)(kFilters >> 4) << 24);
  const int crem = g.C - 32 * (g.Cw - 1);
  P.tail_mask = crem == 32 ? 0xFFFFFFFFu : ((1u << crem) - 1u);
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(binconv_fp4_kernel<2>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemCap);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(binconv_fp4_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)kSmemCap);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  const dim3 grid((unsigned)pl.mtiles, (unsigned)pl.ftiles);
  if (pl.wps == 4) binconv_fp4_kernel<4><<<grid, kThreads, pl.smem, st>>>(P);
  else binconv_fp4_kernel<2><<<grid, kThreads, pl.smem, st>>>(P);
  return cudaGetLastError();
}

cudaError_t read_status_fp4(int *status) {
  cudaError_t e = cudaMemcpyFromSymbol(status, g_status_fp4, sizeof(int));
  if (e == cudaSuccess && *status != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_status_fp4, &zero, sizeof(int));
  }
  return e;
}

#ifdef XNOR_TRACE
extern "C" int xnor_debug_trace(long long *host256) {
  return (int)cudaMemcpyFromSymbol(host256, g_trace, sizeof(long long) * 256);
}
#endif

}  // namespace xnor
