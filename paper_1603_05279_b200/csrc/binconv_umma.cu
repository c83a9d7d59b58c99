// BinConv on the 5th-generation tensor cores (Eq. 11).
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

namespace xnor {

__device__ int g_device_status = 0;

namespace {

constexpr int kProducerWarps = 8;
constexpr int kProducers = 32 * kProducerWarps;
constexpr int kThreads = 32 + kProducers;
constexpr int kTileM = 128;
constexpr int kMaxStages = 6;
constexpr long long kWaitCycles = 1ll << 31;   // about a second

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

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the wait expired or another thread of the
// CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) {
      *abort_flag = 1;
      atomicExch(&g_device_status, (int)XNOR_ERR_TIMEOUT);
      return false;
    }
  }
}

__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// Shared-memory matrix descriptor, no swizzle, K-major: 8-row x 16-byte core
// matrices; lbo = byte distance between the two core matrices along K, sbo =
// byte distance between 8-row groups.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) |
         ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                        uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar) : "memory");
}

// 32 sign bits -> 32 bytes of +1 (0x01) / -1 (0xFF).  Register j holds the
// channels j, j+8, j+16, j+24 of the word (the K order is the same for both
// operands, so any fixed permutation is fine).
__device__ __forceinline__ void expand_word(uint32_t w, uint32_t v[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t t = (w >> j) & 0x01010101u;
    v[j] = 0xFFFFFFFFu - 0xFEu * t;
  }
}

__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c,
                                       uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c),
               "r"(d) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int32_t r[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(kThreads, 2) binconv_umma_kernel(const UmmaParams P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int taps = P.kh * P.kw;
  const uint32_t patch_bytes = (uint32_t)(2 * P.cwc) * P.ppix * 16u;
  const uint32_t stage_bytes = (uint32_t)(2 * P.wps) * P.NT * 16u;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t patch_addr = smem_base;
  const uint32_t stage_addr = patch_addr + patch_bytes;
  uint8_t *ctrl = smem + patch_bytes + (size_t)P.stages * stage_bytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(ctrl);
  // bars: [0,S) full, [S,2S) empty, 2S patch_full, 2S+1 patch_free, 2S+2 accum_full
  const uint32_t bar0 = smem_u32(bars);
  const int S = P.stages;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
  const uint32_t patch_full = bar0 + 8u * (2 * S), patch_free = patch_full + 8u,
                 accum_full = patch_full + 16u;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kMaxStages + 4);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < S; ++s) {
        mbar_init(full_bar(s), kProducerWarps);
        mbar_init(empty_bar(s), 1);
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

  const long long m0 = (long long)blockIdx.x * kTileM;
  const int co0 = blockIdx.y * P.NT;
  const int nchunks = (P.Cw + P.cwc - 1) / P.cwc;

  if (warp == 0) {
    // ------------------------------------------------------------ MMA issuer
    uint32_t it = 0, accumulate = 0;
    bool ok = true;
    for (int cc = 0; cc < nchunks && ok; ++cc) {
      const int cwn = min(P.cwc, P.Cw - cc * P.cwc);
      ok = mbar_wait(patch_full, cc & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      for (int tap = 0; tap < taps && ok; ++tap) {
        const int ky = tap / P.kw, kx = tap - ky * P.kw;
        const uint32_t a_tap = patch_addr + (uint32_t)(ky * P.Wp + kx) * 16u;
        for (int wb = 0; wb < cwn; wb += P.wps, ++it) {
          const int nw = min(P.wps, cwn - wb);
          const int s = it % S;
          ok = mbar_wait(full_bar(s), (it / S) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
            for (int wi = 0; wi < nw; ++wi) {
              const uint64_t ad = make_desc(a_tap + (uint32_t)(2 * (wb + wi)) * P.ppix * 16u,
                                            (uint32_t)P.ppix * 16u, 128u);
              const uint64_t bd = make_desc(stage_addr + s * stage_bytes +
                                                (uint32_t)(2 * wi) * P.NT * 16u,
                                            (uint32_t)P.NT * 16u, 128u);
              umma_i8(tmem_base, ad, bd, P.idesc, accumulate);
              accumulate = 1;
            }
            umma_commit(empty_bar(s));
          }
          __syncwarp();
        }
      }
      if (ok && lane == 0) umma_commit(patch_free);
      __syncwarp();
    }
    if (ok && lane == 0) umma_commit(accum_full);
    __syncwarp();
  } else {
    // ------------------------------------------------------------ producers
    const int pt = tid - 32;
    uint32_t it = 0;
    bool ok = true;
    for (int cc = 0; cc < nchunks && ok; ++cc) {
      const int cw0 = cc * P.cwc;
      const int cwn = min(P.cwc, P.Cw - cw0);
      if (cc > 0) {
        ok = mbar_wait(patch_free, (cc - 1) & 1, abort_flag);
        if (!ok) break;
      }
      // expand the activation patch: item = (word wl, stream pixel q), q fastest
      for (int item = pt; item < P.ppix * cwn; item += kProducers) {
        const int wl = item / P.ppix, q = item - wl * P.ppix;
        const long long sq = m0 + q;
        uint32_t v[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        if (sq < P.L) {
          const long long r = sq / P.Wp;
          const int c = (int)(sq - r * P.Wp);
          const long long n = r / P.Hp;
          const int ry = (int)(r - n * P.Hp);
          if (c >= P.pad && ry >= P.pad) {
            const int cw = cw0 + wl;
            const uint32_t w = __ldg(P.xp + (((size_t)n * P.H + (ry - P.pad)) * P.W + (c - P.pad)) *
                                                P.Cw + cw);
            expand_word(w, v);
            if (cw == P.Cw - 1 && P.tail_mask != 0xFFFFFFFFu) {
#pragma unroll
              for (int j = 0; j < 8; ++j) v[j] &= ((P.tail_mask >> j) & 0x01010101u) * 0xFFu;
            }
          }
        }
        const uint32_t a = patch_addr + (uint32_t)(2 * wl) * P.ppix * 16u + (uint32_t)q * 16u;
        sts128(a, v[0], v[1], v[2], v[3]);
        sts128(a + (uint32_t)P.ppix * 16u, v[4], v[5], v[6], v[7]);
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(patch_full);

      for (int tap = 0; tap < taps && ok; ++tap) {
        for (int wb = 0; wb < cwn; wb += P.wps, ++it) {
          const int nw = min(P.wps, cwn - wb);
          const int s = it % S;
          ok = mbar_wait(empty_bar(s), ((it / S) & 1) ^ 1, abort_flag);
          if (!ok) break;
          if (pt < P.NT) {
            const int co = co0 + pt;
            const uint32_t *src = P.wp + ((size_t)co * taps + tap) * P.Cw + cw0 + wb;
            const uint32_t dst = stage_addr + s * stage_bytes + (uint32_t)pt * 16u;
            for (int wi = 0; wi < nw; ++wi) {
              uint32_t v[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
              if (co < P.Co) expand_word(__ldg(src + wi), v);
              const uint32_t a = dst + (uint32_t)(2 * wi) * P.NT * 16u;
              sts128(a, v[0], v[1], v[2], v[3]);
              sts128(a + (uint32_t)P.NT * 16u, v[4], v[5], v[6], v[7]);
            }
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(full_bar(s));
        }
      }
    }
    // ------------------------------------------------------------ epilogue
    if (ok) ok = mbar_wait(accum_full, 0, abort_flag);
    if (ok) {
      tc_fence_after();
      const int quarter = warp & 3;              // TMEM lanes 32*quarter .. +31
      const int half = (warp - 1) >> 2;          // which half of the column blocks
      const int nblk = P.NT / 16;
      const int b_begin = half == 0 ? 0 : (nblk + 1) / 2;
      const int b_end = half == 0 ? (nblk + 1) / 2 : nblk;
      const long long m = m0 + quarter * 32 + lane;
      bool valid = m < P.L;
      long long n = 0;
      int oy = 0, ox = 0;
      if (valid) {
        const long long r = m / P.Wp;
        ox = (int)(m - r * P.Wp);
        n = r / P.Hp;
        oy = (int)(r - n * P.Hp);
        valid = ox < P.Wo && oy < P.Ho;
      }
      const size_t HoWo = (size_t)P.Ho * P.Wo;
      const size_t pix = (size_t)oy * P.Wo + ox;
      const float kv = valid ? __ldg(P.K + (size_t)n * HoWo + pix) : 0.0f;
      for (int b = b_begin; b < b_end; ++b) {
        int32_t r[16];
        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * 16), r);
        if (valid) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int co = co0 + b * 16 + j;
            if (co < P.Co) {
              const size_t o = ((size_t)n * P.Co + co) * HoWo + pix;
              float v = __fmul_rn(__fmul_rn((float)r[j], kv), __ldg(P.alpha + co));
              if (P.residual) v += P.residual[o];
              P.out[o] = v;
              if (P.acc_out) P.acc_out[o] = r[j];
            }
          }
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

constexpr size_t kSmemBudget = 110 * 1024;   // two CTAs per SM
constexpr size_t kCtrlBytes = 256;

}  // namespace

bool umma_supported(const ConvGeom &g) {
  if (g.stride != 1) return false;
  const int Wp = g.W + g.pad;
  const int halo = (g.kh - 1) * Wp + g.kw - 1;
  const int ppix = (kTileM + halo + 7) / 8 * 8;
  // one channel word of patch plus two minimal weight stages must fit
  const size_t need = (size_t)ppix * 32 + 2 * (size_t)256 * 32 + kCtrlBytes;
  if (need > kSmemBudget) return false;
  if ((size_t)ppix * 16 >= (1u << 18)) return false;
  return true;
}

cudaError_t launch_binconv_umma(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                                const float *K, const float *residual, const ConvGeom &g,
                                float *out, int32_t *acc_out, cudaStream_t st) {
  UmmaParams P;
  P.xp = xp; P.wp = wp; P.alpha = alpha; P.K = K; P.residual = residual;
  P.out = out; P.acc_out = acc_out;
  P.N = g.N; P.C = g.C; P.H = g.H; P.W = g.W; P.Co = g.Co; P.kh = g.kh; P.kw = g.kw;
  P.pad = g.pad; P.Ho = g.Ho; P.Wo = g.Wo; P.Cw = g.Cw;
  P.Hp = g.H + g.pad; P.Wp = g.W + g.pad;
  P.L = (long long)g.N * P.Hp * P.Wp;
  const int halo = (g.kh - 1) * P.Wp + g.kw - 1;
  P.ppix = (kTileM + halo + 7) / 8 * 8;
  const int ntiles = (g.Co + 255) / 256;
  P.NT = (((g.Co + ntiles - 1) / ntiles) + 15) / 16 * 16;
  P.tmem_cols = 32;
  while (P.tmem_cols < P.NT) P.tmem_cols *= 2;
  P.wps = 2;
  const size_t stage_bytes = (size_t)2 * P.wps * P.NT * 16;
  const size_t word_bytes = (size_t)P.ppix * 32;   // patch bytes per channel word
  int stages = 4, cwc = 0;
  for (; stages >= 2; --stages) {
    const size_t left = kSmemBudget - kCtrlBytes - stages * stage_bytes;
    cwc = (int)(left / word_bytes);
    if (cwc >= g.Cw) break;
  }
  if (stages < 2) {   // the whole channel range does not fit: chunk it, keep 3 stages
    stages = 3;
    cwc = (int)((kSmemBudget - kCtrlBytes - stages * stage_bytes) / word_bytes);
  }
  if (cwc > g.Cw) cwc = g.Cw;
  if (cwc < 1) return cudaErrorInvalidValue;
  P.cwc = cwc;
  P.stages = stages;
  P.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.NT >> 3) << 17) |
            ((uint32_t)(kTileM >> 4) << 24);
  const int crem = g.C - 32 * (g.Cw - 1);
  P.tail_mask = crem == 32 ? 0xFFFFFFFFu : ((1u << crem) - 1u);
  const size_t smem = (size_t)2 * cwc * P.ppix * 16 + stages * stage_bytes + kCtrlBytes;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(binconv_umma_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemBudget);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  const long long mtiles = (P.L + kTileM - 1) / kTileM;
  const dim3 grid((unsigned)mtiles, (unsigned)ntiles);
  binconv_umma_kernel<<<grid, kThreads, smem, st>>>(P);
  return cudaGetLastError();
}

cudaError_t read_device_status(int *status, cudaStream_t st) {
  cudaError_t e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(status, g_device_status, sizeof(int));
  if (e != cudaSuccess) return e;
  if (*status != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
  }
  return e;
}

}  // namespace xnor
