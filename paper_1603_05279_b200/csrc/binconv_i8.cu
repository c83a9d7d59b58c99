// BinConv on the 5th-generation tensor cores with int8 operands (Eq. 11).
// Kept beside the fp4 kernel as the measured alternative: same structure, half
// the tensor-core rate and twice the shared-memory bytes per 1-bit MAC.
//
// sign(I) (*) sign(W) is an exact integer contraction, so it runs as an
// implicit GEMM with +-1/0 int8 operands and int32 accumulators in tensor
// memory (tcgen05.mma kind::i8).  HBM only ever sees the 1-bit packed words;
// each CTA expands what it needs into shared memory:
//
//  * Activations.  All images are laid out (virtually) as one long stream of
//    pixels: every image row is preceded by `pad` zero pixels and every image
//    by `pad` zero rows, so row width is Wp = W + pad and image height
//    Hp = H + pad; the zeros to the right of a row / below an image are the
//    ones that precede the next row / image.  With GEMM row m = stream index
//    of the output pixel, filter tap (ky,kx) reads stream pixel
//    m + ky*Wp + kx: a pure shift.  A CTA owns 128 consecutive m and expands
//    the 128 + (kh-1)*Wp + (kw-1) stream pixels it touches ONCE; every tap's
//    A operand is then the same shared-memory patch at a shifted start
//    address (no-swizzle K-major layout: 8 pixels x 16 channel-bytes per core
//    matrix, pixels contiguous).  Zero pixels and the channel tail expand to
//    byte 0, so padded taps contribute exactly 0 with no mask or correction.
//    Stream positions that are padding produce junk rows that are never stored.
//  * Weights.  Streamed through a ring of shared-memory stages, one (tap, up
//    to 64 channels) slab per stage, expanded from bits by the producer warps.
//
// Warp 0 issues the MMAs; warps 1..8 expand operands and then run the
// epilogue (tcgen05.ld, * K * alpha, + residual, coalesced NCHW stores).
// Every wait is bounded: on expiry the CTA records XNOR_ERR_TIMEOUT in a
// device status word, stops issuing work, frees its tensor memory and exits.
#include "common.cuh"
#include "umma_common.cuh"

namespace xnor {

__device__ int g_status_i8 = 0;

namespace {

using namespace umma;

constexpr int kProducerWarps = 8;
constexpr int kProducers = 32 * kProducerWarps;
constexpr int kThreads = 32 + kProducers;
constexpr int kTileM = 128;
constexpr int kMaxStages = 6;
constexpr int kMaxWps = 4;       // channel words per weight stage (one MMA of K = 32 each)
constexpr int kPrefetch = 4;     // weight stages whose packed words are in flight
constexpr int kMaxChunkWords = 16;  // channel words of the patch resident at a time, upper bound
constexpr size_t kCtrlBytes = 256;

struct UmmaParams {
  const uint32_t *xp, *wp;
  const float *alpha, *K, *residual;
  float *out;
  int32_t *acc_out;
  int N, C, H, W, Co, kh, kw, pad, Ho, Wo, Cw, Hp, Wp;
  long long L;      // stream length N*Hp*Wp
  int ppix;         // stream pixels staged per CTA (128 + halo, rounded up to 8)
  int NT;           // filters per CTA, multiple of 16
  int tmem_cols;    // power of two >= NT
  int cwc;          // channel words per patch chunk
  int wps;          // channel words per weight stage
  int stages;
  uint32_t idesc;
  uint32_t tail_mask;  // bits of real channels in the last word (all ones if C % 32 == 0)
};

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                        uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// Operand encodings.  Bit j of every byte of a packed word (channels j, j+8,
// j+16, j+24) lands in register j of the 32 expanded bytes; both operands use
// the same order, so the K order is consistent.
//
// Weights take ONE logic op per register: byte = beta * 2^j (beta = sign bit,
// 0 or 1) for j = 0..6 is just `w & (0x01010101 << j)`; bit 7 is moved down to
// beta * 64.  Activations carry the compensating power of two and the sign:
// byte = a * 2^(6-j) (a = +-1; 0 for padding and for the channel tail), and
// a * 1 for j = 7.  Every product is 64 * a * beta, so the tensor core returns
// D = 64 * sum(a * beta).  With sign(W) = 2 beta - 1 the wanted sum is
//   sum(a * sign(W)) = D / 32 - S,   S = sum of a over the window,
// and S is a box sum of per-pixel values (2 popcount - channels) that the
// activation expansion leaves in shared memory.  All of it is exact integer
// arithmetic (|D| <= 64 * C_in * k_h * k_w < 2^31).
__device__ __forceinline__ void expand_weights(uint32_t w, uint32_t v[8]) {
#pragma unroll
  for (int j = 0; j < 7; ++j) v[j] = w & (0x01010101u << j);
  v[7] = (w >> 1) & 0x40404040u;
}

__device__ __forceinline__ void expand_activations(uint32_t w, uint32_t v[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t sc = j < 7 ? (64u >> j) : 1u;                // |byte value|
    const uint32_t t = (w >> j) & 0x01010101u;                  // sign bit per byte
    v[j] = (256u - sc) * 0x01010101u - t * (256u - 2u * sc);    // bit ? +sc : -sc, no borrows
  }
}

// NT_CT: filters per CTA when known at compile time (0 = read P.NT); WPS: channel
// words per weight stage.  Both only remove address arithmetic and predicates.
template <int NT_CT, int WPS>
__global__ void __launch_bounds__(kThreads, 2) binconv_i8_kernel(const UmmaParams P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int taps = P.kh * P.kw;
  const int NT = NT_CT ? NT_CT : P.NT;
  const uint32_t patch_bytes = (uint32_t)(2 * P.cwc) * P.ppix * 16u;
  const uint32_t stage_bytes = (uint32_t)(2 * WPS) * NT * 16u;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t patch_addr = smem_base;
  const uint32_t stage_addr = patch_addr + patch_bytes;
  uint8_t *ctrl = smem + patch_bytes + (size_t)P.stages * stage_bytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(ctrl);
  // bars: [0,S) full, [S,2S) empty, 2S patch_full, 2S+1 patch_free, 2S+2 accum_full
  const uint32_t bar0 = smem_u32(bars);
  const int S = P.stages;
  const uint32_t patch_full = bar0 + 8u * (2 * S), patch_free = patch_full + 8u,
                 accum_full = patch_full + 16u;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kMaxStages + 4);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  int *pix_sum = reinterpret_cast<int *>(ctrl + kCtrlBytes);   // [ppix] sum over channels of a
  float *alpha_sm = reinterpret_cast<float *>(pix_sum + P.ppix);  // [NT], 16-byte aligned

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
                 ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)P.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const uint32_t m0 = blockIdx.x * (uint32_t)kTileM;
  const int co0 = blockIdx.y * NT;
  const int nchunks = (P.Cw + P.cwc - 1) / P.cwc;
  const uint32_t a_lbo = (uint32_t)P.ppix * 16u, b_lbo = (uint32_t)NT * 16u;

  if (warp == 0) {
    // ------------------------------------------------------------ MMA issuer
    uint32_t accumulate = 0, ph = 0;
    int s = 0;
    bool ok = true;
    for (int cc = 0; cc < nchunks && ok; ++cc) {
      const int cwn = min(P.cwc, P.Cw - cc * P.cwc);
      ok = mbar_wait(patch_full, cc & 1, abort_flag, &g_status_i8);
      if (!ok) break;
      tc_fence_after();
      int kx = 0;
      uint32_t a_tap = patch_addr;                       // + (ky*Wp + kx) * 16
      for (int tap = 0; tap < taps && ok; ++tap) {
        for (int wb = 0; wb < cwn; wb += WPS) {
          const int nw = min(WPS, cwn - wb);
          ok = mbar_wait(bar0 + 8u * s, ph, abort_flag, &g_status_i8);
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
            uint32_t a_addr = a_tap + (uint32_t)(2 * wb) * a_lbo;
            uint32_t b_addr = stage_addr + s * stage_bytes;
            for (int wi = 0; wi < nw; ++wi) {
              umma_i8(tmem_base, make_desc(a_addr, a_lbo, 128u), make_desc(b_addr, b_lbo, 128u),
                      P.idesc, accumulate);
              accumulate = 1;
              a_addr += 2u * a_lbo;
              b_addr += 2u * b_lbo;
            }
            umma_commit(bar0 + 8u * (S + s));
          }
          __syncwarp();
          if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (++kx == P.kw) { kx = 0; a_tap += (uint32_t)(P.Wp - P.kw + 1) * 16u; }
        else a_tap += 16u;
      }
      if (ok && lane == 0) umma_commit(patch_free);
      __syncwarp();
    }
    if (ok && lane == 0) umma_commit(accum_full);
    __syncwarp();
  } else {
    // ------------------------------------------------------------ producers
    const int pt = tid - 32;
    uint32_t ph = 1;          // parity to wait for on the empty barriers
    int s = 0;
    bool ok = true;
    const int crem = P.C - 32 * (P.Cw - 1);
    for (int cc = 0; cc < nchunks && ok; ++cc) {
      const int cw0 = cc * P.cwc;
      const int cwn = min(P.cwc, P.Cw - cw0);
      if (cc > 0) {
        ok = mbar_wait(patch_free, (cc - 1) & 1, abort_flag, &g_status_i8);
        if (!ok) break;
      }
      // expand the activation patch: one thread per stream pixel, all channel words of
      // the chunk; every global load is issued before the first expansion
      if (cc == 0)
        for (int i = pt; i < NT; i += kProducers)
          alpha_sm[i] = co0 + i < P.Co ? __ldg(P.alpha + co0 + i) : 0.0f;
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
          if (wl < cwn) {
            uint32_t v[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
            if (src != nullptr) {
              expand_activations(pw[wl], v);
              int nreal = 32;
              if (cw0 + wl == P.Cw - 1 && crem != 32) {
                nreal = crem;
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] &= ((P.tail_mask >> j) & 0x01010101u) * 0xFFu;
              }
              psum += 2 * __popc(pw[wl]) - nreal;
            }
            sts128(a, v[0], v[1], v[2], v[3]);
            sts128(a + a_lbo, v[4], v[5], v[6], v[7]);
            a += 2u * a_lbo;
          }
        }
        pix_sum[q] += psum;
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(patch_full);

      // weight stages of this chunk in the issuer's order (tap outer, words inner).
      // kPrefetch register sets hold the packed words of the next stages; a set is
      // refilled right after it is expanded, so a load has kPrefetch stages to land.
      const int co = co0 + pt;
      const bool row_live = pt < NT && co < P.Co;
      const int f_co = row_live ? co : 0;
      int f_word = cw0;                               // word index of (tap f_tap, word 0 of the chunk)
      int f_wb = 0, f_tap = row_live ? 0 : taps;     // dead rows never fetch
      uint32_t pf[kPrefetch][WPS];
      auto fetch = [&](uint32_t dst[WPS]) {
        if (f_tap < taps) {
#pragma unroll
          for (int wi = 0; wi < WPS; ++wi)
            dst[wi] = f_wb + wi < cwn
                          ? __ldg(P.wp + packed_weight_index(P.Co, f_co, f_word + f_wb + wi)) : 0u;
          f_wb += WPS;
          if (f_wb >= cwn) { f_wb = 0; ++f_tap; f_word += P.Cw; }
        } else {
#pragma unroll
          for (int wi = 0; wi < WPS; ++wi) dst[wi] = 0u;
        }
      };
#pragma unroll
      for (int d = 0; d < kPrefetch; ++d) fetch(pf[d]);
      const uint32_t row_addr = stage_addr + (uint32_t)pt * 16u;
      int tap = 0, wb = 0;
      while (tap < taps && ok) {
#pragma unroll
        for (int d = 0; d < kPrefetch; ++d) {
          if (tap < taps && ok) {
            ok = mbar_wait(bar0 + 8u * (S + s), ph, abort_flag, &g_status_i8);
            if (ok) {
              if (pt < NT) {
                const uint32_t a = row_addr + s * stage_bytes;
                const int nw = cwn - wb;           // >= WPS except in a ragged last stage
#pragma unroll
                for (int wi = 0; wi < WPS; ++wi) {
                  if (wi == 0 || wi < nw) {
                    uint32_t v[8];
                    expand_weights(pf[d][wi], v);      // 0 for rows beyond C_out
                    sts128(a + (uint32_t)(2 * wi) * b_lbo, v[0], v[1], v[2], v[3]);
                    sts128(a + (uint32_t)(2 * wi + 1) * b_lbo, v[4], v[5], v[6], v[7]);
                  }
                }
              }
              fence_proxy_async();
              __syncwarp();
              if (lane == 0) mbar_arrive(bar0 + 8u * s);
              if (++s == S) { s = 0; ph ^= 1u; }
              wb += WPS;
              if (wb >= cwn) { wb = 0; ++tap; }
              fetch(pf[d]);
            }
          }
        }
      }
    }
    // ------------------------------------------------------------ epilogue
    if (ok) ok = mbar_wait(accum_full, 0, abort_flag, &g_status_i8);
    if (ok) {
      tc_fence_after();
      const int quarter = warp & 3;              // TMEM lanes 32*quarter .. +31
      const int half = (warp - 1) >> 2;          // which half of the column blocks
      const int nblk = NT / 16;
      const int b_begin = half == 0 ? 0 : (nblk + 1) / 2;
      const int b_end = half == 0 ? (nblk + 1) / 2 : nblk;
      const int lm = quarter * 32 + lane;
      const uint32_t m = m0 + (uint32_t)lm;
      bool valid = m < (uint32_t)P.L;
      uint32_t n = 0;
      int oy = 0, ox = 0;
      if (valid) {
        const uint32_t r = m / (uint32_t)P.Wp;
        ox = (int)(m - r * (uint32_t)P.Wp);
        n = r / (uint32_t)P.Hp;
        oy = (int)(r - n * (uint32_t)P.Hp);
        valid = ox < P.Wo && oy < P.Ho;
      }
      int wsum = 0;                               // S: sum of a over the window of pixel m
      if (valid) {
        for (int ky = 0; ky < P.kh; ++ky)
          for (int kx = 0; kx < P.kw; ++kx) wsum += pix_sum[lm + ky * P.Wp + kx];
      }
      const size_t HoWo = (size_t)P.Ho * P.Wo;
      const size_t pix = (size_t)oy * P.Wo + ox;
      // out = (D/32 - S) * K * alpha, evaluated as float(D - 32 S) * (K/32) * alpha: the
      // power-of-two factors move exactly, and |D - 32 S| < 2^24 so the conversion is exact
      const float kvs = valid ? __ldg(P.K + (size_t)n * HoWo + pix) * 0.03125f : 0.0f;
      const int wsum32 = wsum * 32;
      const size_t o0 = ((size_t)n * P.Co + co0 + b_begin * 16) * HoWo + pix;
      float *optr = P.out + o0;
      const bool plain = P.residual == nullptr && P.acc_out == nullptr;
      const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
      auto emit = [&](int b, const int32_t r[16]) {
        if (valid) {
          if (plain && co0 + b * 16 + 16 <= P.Co) {
            float *p = optr;
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
              const float4 al = *reinterpret_cast<const float4 *>(alpha_sm + b * 16 + j4 * 4);
              const float a4[4] = {al.x, al.y, al.z, al.w};
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) {
                *p = __fmul_rn(__fmul_rn((float)(r[j4 * 4 + jj] - wsum32), kvs), a4[jj]);
                p += HoWo;
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int co = co0 + b * 16 + j;
              if (co < P.Co) {
                const size_t o = (size_t)(optr - P.out) + (size_t)j * HoWo;
                float v = __fmul_rn(__fmul_rn((float)(r[j] - wsum32), kvs), alpha_sm[b * 16 + j]);
                if (P.residual) v += P.residual[o];
                P.out[o] = v;
                if (P.acc_out) P.acc_out[o] = (r[j] - wsum32) >> 5;
              }
            }
          }
          optr += 16 * HoWo;
        }
      };
      // two register sets: the load of the next 16 columns is in flight while the
      // current 16 are scaled and stored
      int32_t ra[16], rb[16];
      if (b_begin < b_end) {
        tmem_ld16(t_lane + (uint32_t)(b_begin * 16), ra);
        tmem_wait16(ra);
      }
      for (int b = b_begin; b < b_end; b += 2) {
        if (b + 1 < b_end) tmem_ld16(t_lane + (uint32_t)((b + 1) * 16), rb);
        emit(b, ra);
        if (b + 1 < b_end) {
          tmem_wait16(rb);
          if (b + 2 < b_end) tmem_ld16(t_lane + (uint32_t)((b + 2) * 16), ra);
          emit(b + 1, rb);
          if (b + 2 < b_end) tmem_wait16(ra);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"((uint32_t)P.tmem_cols) : "memory");
  }
}

constexpr size_t kSmemBudget = 115000;   // two CTAs per SM

struct Plan {
  int ppix, NT, ntiles, tmem_cols, cwc, wps, stages;
  size_t smem;
  bool ok;
};

Plan make_plan(const ConvGeom &g) {
  Plan p{};
  p.ok = false;
  if (g.stride != 1) return p;
  const int Wp = g.W + g.pad, Hp = g.H + g.pad;
  if ((long long)g.N * Hp * Wp >= (1ll << 31) - kTileM) return p;
  const int halo = (g.kh - 1) * Wp + g.kw - 1;
  p.ppix = (kTileM + halo + 7) / 8 * 8;
  if ((size_t)p.ppix * 16 >= (1u << 18)) return p;
  p.ntiles = (g.Co + 255) / 256;
  p.NT = (((g.Co + p.ntiles - 1) / p.ntiles) + 15) / 16 * 16;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.NT) p.tmem_cols *= 2;
  const size_t fixed = kCtrlBytes + (size_t)p.ppix * sizeof(int) + (size_t)p.NT * sizeof(float);
  const size_t word_bytes = (size_t)p.ppix * 32;            // patch bytes per channel word
  const size_t max_patch_words = kMaxChunkWords;
  // whole channel range resident: pick the stage width that needs the fewest stage steps
  long best_steps = -1;
  if ((size_t)g.Cw <= max_patch_words) {
    for (int wps = kMaxWps; wps >= 1; --wps) {
      const size_t stage_bytes = (size_t)2 * wps * p.NT * 16;
      if (fixed + word_bytes * g.Cw + 3 * stage_bytes > kSmemBudget) continue;
      int stages = (int)((kSmemBudget - fixed - word_bytes * g.Cw) / stage_bytes);
      if (stages > kMaxStages) stages = kMaxStages;
      // stage steps per tap, with a small penalty per barrier round trip
      const long steps = (g.Cw + wps - 1) / wps * (long)(wps * 4 + 1);
      if (best_steps < 0 || steps < best_steps) {
        best_steps = steps; p.wps = wps; p.stages = stages; p.cwc = g.Cw;
      }
    }
  }
  if (best_steps < 0) {   // chunk the channels: 3 stages of 2 words, the rest for the patch
    p.wps = 2; p.stages = 3;
    const size_t stage_bytes = (size_t)2 * p.wps * p.NT * 16;
    if (fixed + 3 * stage_bytes + word_bytes > kSmemBudget) return p;
    size_t cwc = (kSmemBudget - fixed - 3 * stage_bytes) / word_bytes;
    if (cwc > max_patch_words) cwc = max_patch_words;
    if (cwc > (size_t)g.Cw) cwc = g.Cw;
    p.cwc = (int)cwc;
  }
  p.smem = (size_t)p.cwc * word_bytes + (size_t)p.stages * 2 * p.wps * p.NT * 16 + fixed;
  p.ok = true;
  return p;
}

}  // namespace

bool umma_i8_supported(const ConvGeom &g) { return make_plan(g).ok; }

cudaError_t launch_binconv_i8(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                                const float *K, const float *residual, const ConvGeom &g,
                                float *out, int32_t *acc_out, cudaStream_t st) {
  const Plan pl = make_plan(g);
  if (!pl.ok) return cudaErrorInvalidValue;
  UmmaParams P;
  P.xp = xp; P.wp = wp; P.alpha = alpha; P.K = K; P.residual = residual;
  P.out = out; P.acc_out = acc_out;
  P.N = g.N; P.C = g.C; P.H = g.H; P.W = g.W; P.Co = g.Co; P.kh = g.kh; P.kw = g.kw;
  P.pad = g.pad; P.Ho = g.Ho; P.Wo = g.Wo; P.Cw = g.Cw;
  P.Hp = g.H + g.pad; P.Wp = g.W + g.pad;
  P.L = (long long)g.N * P.Hp * P.Wp;
  P.ppix = pl.ppix; P.NT = pl.NT; P.tmem_cols = pl.tmem_cols;
  P.cwc = pl.cwc; P.wps = pl.wps; P.stages = pl.stages;
  P.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.NT >> 3) << 17) |
            ((uint32_t)(kTileM >> 4) << 24);
  const int crem = g.C - 32 * (g.Cw - 1);
  P.tail_mask = crem == 32 ? 0xFFFFFFFFu : ((1u << crem) - 1u);
  using KernelFn = void (*)(const UmmaParams);
  static const KernelFn table[5][kMaxWps] = {
#define XNOR_ROW(NT) {binconv_i8_kernel<NT, 1>, binconv_i8_kernel<NT, 2>, \
                      binconv_i8_kernel<NT, 3>, binconv_i8_kernel<NT, 4>}
      XNOR_ROW(0), XNOR_ROW(64), XNOR_ROW(128), XNOR_ROW(192), XNOR_ROW(256)
#undef XNOR_ROW
  };
  static bool attr_set = false;
  if (!attr_set) {
    for (int i = 0; i < 5; ++i)
      for (int j = 0; j < kMaxWps; ++j) {
        cudaError_t e = cudaFuncSetAttribute(table[i][j],
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemBudget);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
      }
    attr_set = true;
  }
  const int row = (P.NT % 64 == 0) ? P.NT / 64 : 0;
  const long long mtiles = (P.L + kTileM - 1) / kTileM;
  const dim3 grid((unsigned)mtiles, (unsigned)pl.ntiles);
  table[row][P.wps - 1]<<<grid, kThreads, pl.smem, st>>>(P);
  return cudaGetLastError();
}

cudaError_t read_status_i8(int *status) {
  cudaError_t e = cudaMemcpyFromSymbol(status, g_status_i8, sizeof(int));
  if (e == cudaSuccess && *status != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_status_i8, &zero, sizeof(int));
  }
  return e;
}

}  // namespace xnor
