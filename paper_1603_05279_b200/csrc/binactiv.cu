// BatchNorm affine + BinActiv (Section 3.2): sign bits packed along channels,
// A = channel mean of |y|, then K = box filter of zero-padded A at the
// convolution's output positions.
#include <algorithm>

#include "kbit.cuh"
#include "umma_common.cuh"

namespace xnor {

namespace {

constexpr int kPix = 32;        // pixels per group: one warp wide
constexpr int kWarps = 8;       // warps per block
constexpr int kTileFloats = 32 * kPix;                 // one (32 channels x 32 pixels) tile
constexpr int kBufsPerWarp = 2;

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// Persistent blocks of 8 warps.  A task is (group of 32 consecutive pixels, flat over n,h,w;
// 32-channel word): lane = pixel, so one channel of a task is a contiguous 128-byte run of
// x.  The G warps of a pixel group take words g, g + G, ...; a block works on 8 / G pixel
// groups at a time.  G = 1 (a warp packs whole pixel groups, no block-wide step) when there
// are enough pixel groups to fill the GPU, else min(Cw, 8).  Input goes global -> shared with 4-byte cp.async, two tiles
// per warp in flight while a third is processed, so the bytes in flight per SM (what HBM
// bandwidth needs) do not depend on how the compiler schedules loads against their uses.
// Packed words are staged and written as contiguous runs; A is reduced over the warps of a
// pixel group in a fixed order.
template <bool kHasBN, bool kVec16>
__global__ void __launch_bounds__(32 * kWarps)
binactiv_pack_kernel(const float *__restrict__ x, const float *__restrict__ scale,
                     const float *__restrict__ shift, long long total_pix, int C, int HW, int Cw,
                     int G, int PG, uint32_t *__restrict__ x_packed, float *__restrict__ A) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  float *stage = reinterpret_cast<float *>(smem_raw);                      // [warp][buf][32][32]
  float2 *bn = reinterpret_cast<float2 *>(stage + kWarps * kBufsPerWarp * kTileFloats);  // [Cw*32]
  uint32_t *words = reinterpret_cast<uint32_t *>(bn + (kHasBN ? Cw * 32 : 0));  // [PG][32][Cw]
  float *sabs = reinterpret_cast<float *>(words + PG * kPix * Cw);          // [PG][G][32]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int pgl = warp / G, g = warp - pgl * G;
  const bool active = pgl < PG;
  if (kHasBN) {
    for (int c = threadIdx.x; c < Cw * 32; c += 32 * kWarps)
      bn[c] = c < C ? make_float2(__ldg(scale + c), __ldg(shift + c)) : make_float2(0.0f, 0.0f);
  }
  __syncthreads();

  const long long ngroups = (total_pix + kPix - 1) / kPix;
  const long long nbatches = (ngroups + PG - 1) / PG;
  const int nw = active ? (Cw - g + G - 1) / G : 0;        // words of this warp per pixel group
  float *my_stage = stage + warp * kBufsPerWarp * kTileFloats;

  // cp.async of one task's tile; always commits a group so that the group count is uniform
  constexpr bool vec16 = kVec16;          // every 4-pixel chunk of x is 16-byte aligned (HW % 4 == 0)
  auto issue = [&](long long batch, int k, int buf) {
    if (batch < nbatches && k < nw && vec16) {
      // a lane copies 4 consecutive pixels of one channel: 8 copies per tile instead of 32
      const long long gp = (batch * PG + pgl) * kPix + 4 * (lane & 7);
      const int c0 = (g + k * G) * 32;
      if (gp < total_pix) {                 // total_pix is a multiple of 4 here
        const long long n = gp / HW;
        const int p = (int)(gp - n * HW);
        const int ch = lane >> 3;           // + 4 q
        const float *src = x + ((size_t)n * C + c0 + ch) * HW + p;
        uint32_t dst = smem_addr(my_stage + buf * kTileFloats + ch * kPix + 4 * (lane & 7));
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          if (c0 + ch + 4 * q < C)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                         ::"r"(dst + (uint32_t)q * 4 * kPix * 4), "l"(src + (size_t)q * 4 * HW)
                         : "memory");
        }
      }
    } else if (batch < nbatches && k < nw) {
      const long long gp = (batch * PG + pgl) * kPix + lane;
      if (gp < total_pix) {
        const long long n = gp / HW;
        const int p = (int)(gp - n * HW);
        const int c0 = (g + k * G) * 32;
        const float *src = x + ((size_t)n * C + c0) * HW + p;
        uint32_t dst = smem_addr(my_stage + buf * kTileFloats + lane);
        const int nc = min(32, C - c0);
        if (nc == 32) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;"
                         ::"r"(dst + (uint32_t)j * kPix * 4), "l"(src + (size_t)j * HW) : "memory");
        } else {
          for (int j = 0; j < nc; ++j)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;"
                         ::"r"(dst + (uint32_t)j * kPix * 4), "l"(src + (size_t)j * HW) : "memory");
        }
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  // this warp's tasks in order: (batch, k) with k = 0 .. nw-1
  long long fb = blockIdx.x;      // batch of the next task to fetch
  int fk = 0, fbuf = 0;
  auto advance_fetch = [&]() {
    if (++fk >= nw) { fk = 0; fb += gridDim.x; }
    fbuf ^= 1;
  };
  issue(fb, fk, fbuf); advance_fetch();
  issue(fb, fk, fbuf); advance_fetch();

  int buf = 0;
  for (long long batch = blockIdx.x; batch < nbatches; batch += gridDim.x) {
    const long long gp0 = (batch * PG + pgl) * kPix;
    const bool live = active && gp0 + lane < total_pix;
    float asum = 0.0f;
    for (int k = 0; k < nw; ++k) {
      asm volatile("cp.async.wait_group 1;" ::: "memory");   // the older of the two tiles landed
      __syncwarp();                      // ... for every lane: a lane reads what other lanes copied
      const int cw = g + k * G;
      const int c0 = cw * 32;
      const float *t = my_stage + buf * kTileFloats + lane;
      uint32_t word = 0u;
      float part = 0.0f;
      if (live) {
        const float2 *ss = bn + c0;
        if (c0 + 32 <= C) {
          // two interleaved sums keep the additions from forming one long dependent chain
          float p0 = 0.0f, p1 = 0.0f;
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float y0 = t[j * kPix], y1 = t[(j + 1) * kPix];
            if (kHasBN) {
              y0 = __fmaf_rn(ss[j].x, y0, ss[j].y);
              y1 = __fmaf_rn(ss[j + 1].x, y1, ss[j + 1].y);
            }
            if (y0 >= 0.0f) word |= 1u << j;
            if (y1 >= 0.0f) word |= 2u << j;
            p0 += fabsf(y0);
            p1 += fabsf(y1);
          }
          part = p0 + p1;
        } else {
          for (int j = 0; c0 + j < C; ++j) {
            float y = t[j * kPix];
            if (kHasBN) y = __fmaf_rn(ss[j].x, y, ss[j].y);
            if (y >= 0.0f) word |= 1u << j;
            part += fabsf(y);
          }
        }
      }
      asum += part;
      words[(pgl * kPix + lane) * Cw + cw] = word;
      __syncwarp();                      // every lane is done reading the tile before it is refilled
      issue(fb, fk, buf); advance_fetch();                   // refill the tile just consumed
      buf ^= 1;
    }
    if (G == 1) {
      // one warp owns the pixel group: no block-wide step, the warp's stream of tiles never stops
      if (live) A[gp0 + lane] = asum / (float)C;
      __syncwarp();
      long long npix = total_pix - gp0;
      if (npix > kPix) npix = kPix;
      if (npix > 0) {
        uint32_t *dst = x_packed + (size_t)gp0 * Cw;
        const uint32_t *srcw = words + pgl * kPix * Cw;
        for (int i = lane; i < (int)npix * Cw; i += 32) dst[i] = srcw[i];
      }
      __syncwarp();
      continue;
    }
    if (active) sabs[(pgl * G + g) * kPix + lane] = asum;
    __syncthreads();
    if (active && g == 0 && live) {
      float sum = 0.0f;
      for (int i = 0; i < G; ++i) sum += sabs[(pgl * G + i) * kPix + lane];
      A[gp0 + lane] = sum / (float)C;
    }
    // the PG pixel groups of a batch are consecutive: one contiguous run of words
    const long long bp0 = batch * PG * kPix;
    long long npix = total_pix - bp0;
    if (npix > PG * kPix) npix = PG * kPix;
    uint32_t *dst = x_packed + (size_t)bp0 * Cw;
    for (int i = threadIdx.x; i < (int)npix * Cw; i += 32 * kWarps) dst[i] = words[i];
    __syncthreads();
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------------------
// Whole-image variant for planes whose size is not a multiple of four pixels.  There a
// channel's 128-byte run of 32 pixels starts on a 4-byte boundary only, and fetching the
// runs one by one is bounded by the number of memory instructions, not by HBM.  An image
// (C x H x W floats) is contiguous and, with C % 4 == 0, starts on a 16-byte boundary: a block
// streams it as chunks of `cc` whole channel planes with one bulk copy each (a dedicated warp
// issues them, `nbuf` chunks deep, also across images), and the eight consumer warps pack out
// of shared memory: unit = (group of 32 pixels, 8 channels), lane = pixel, so the eight
// values of a lane are `H W` words apart (no bank conflicts).  A unit yields one byte of the
// packed words and a partial sum of |y|.  The pixel groups (and, on small planes, the channel
// blocks) of a warp are the same for every chunk, so a lane keeps the |y| sums of its pixels in
// registers through the whole image: no atomics, a fixed order.  At the end of an image the
// block has A of the whole image in shared memory, so K (the box filter of A) is computed
// here too, and the packed words leave as one contiguous run.
constexpr int kImgWarps = 16;
constexpr int kImgThreads = 32 * (kImgWarps + 1);
constexpr int kImgMaxBufs = 4;
constexpr int kImgRounds = 4;                    // pixel groups per warp: planes of up to 1024 pixels

__device__ int g_status_act = 0;

struct ImgParams {
  const float *x, *scale, *shift;
  uint32_t *x_packed;
  float *A, *K;
  int N, C, H, W, Cw;
  int cc, nbuf;                    // channels per chunk (multiple of 8, divides C), chunks in flight
  uint32_t chunk_bytes;            // cc * H * W * 4, a multiple of 16
  uint32_t off_buf, off_words, off_apart, off_aimg, off_bn;   // byte offsets in shared memory
  int kh, kw, stride, pad, Ho, Wo, valid_taps;
  int kbits;                       // k-bit mode: bit planes of the level index (x_packed = [k][N][H][W][Cw])
};

__device__ __forceinline__ float lds_f(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 lds_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

// Barrier over the consumer warps with a bounded wait (a plain bar.sync would wait for ever
// for a warp that gave up).
__device__ __forceinline__ bool img_sync(uint32_t bar, uint32_t &phase, int lane, volatile int *abort_flag) {
  __syncwarp();
  if (lane == 0) umma::mbar_arrive(bar);
  const bool ok = umma::mbar_wait(bar, phase, abort_flag, &g_status_act);
  phase ^= 1u;
  return __all_sync(0xFFFFFFFFu, ok);
}

// kKbit: q_k in place of sign (see binactiv_pack_kbit_kernel below for the rule): a unit then
// yields one byte of each of the k bit planes, staged plane by plane.
template <bool kHasBN, int KS, bool kKbit>
__global__ void __launch_bounds__(kImgThreads, 2)
binactiv_image_kernel(const __grid_constant__ ImgParams P) {
  using namespace umma;
  extern __shared__ __align__(128) uint8_t smem_img[];
  // [0, 64): full barriers, [64, 128): empty barriers, 128: consumer barrier, 136: abort flag
  const uint32_t base = smem_u32(smem_img);
  const uint32_t full = base, empty = base + 8u * kImgMaxBufs, cbar = base + 16u * kImgMaxBufs;
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_img + 16 * kImgMaxBufs + 8);
  uint8_t *wbytes = smem_img + P.off_words;                               // [HW][Cw * 4]
  float *apart = reinterpret_cast<float *>(smem_img + P.off_apart);       // [warps per pixel group][HW]
  float *aimg = reinterpret_cast<float *>(smem_img + P.off_aimg);         // [HW]
  float2 *bn = reinterpret_cast<float2 *>(smem_img + P.off_bn);           // [C]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int HW = P.H * P.W, nsub = P.cc >> 3, nchunks = P.C / P.cc;
  const int npg = (HW + 31) >> 5;
  const int nplanes = kKbit ? P.kbits : 1;
  const uint32_t plane_bytes = (uint32_t)HW * (uint32_t)P.Cw * 4u;      // staged words of one bit plane
  __shared__ float tau[kKbit ? 128 : 1];     // decision points tau[j], j = 1 .. 2^k - 1
  if (kKbit) {
    const int levels = (1 << P.kbits) - 1;
    for (int j = 1 + tid; j <= levels; j += kImgThreads)
      tau[j] = (float)((double)(2 * j - 1) / (double)levels - 1.0);
  }

  const int my_images = ((int)blockIdx.x < P.N) ? (P.N - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  const long long total = (long long)my_images * nchunks;
  // producer state: next chunk to issue (image pn, chunk pch of it) into buffer pb
  long long q = 0;
  int pn = blockIdx.x, pch = 0, pb = 0;
  uint32_t eph = 1u;                   // parity of an empty barrier's phase before its first completion
  auto issue_chunk = [&]() {
    const float *src = P.x + ((size_t)pn * P.C + (size_t)pch * P.cc) * HW;
    mbar_arrive_expect_tx(full + 8u * pb, P.chunk_bytes);
    bulk_copy_g2s(base + P.off_buf + (uint32_t)pb * P.chunk_bytes, src, P.chunk_bytes, full + 8u * pb);
    if (++pch == nchunks) { pch = 0; pn += gridDim.x; }
    if (++pb == P.nbuf) { pb = 0; eph ^= 1u; }
  };
  const bool producer = warp == kImgWarps && lane == 0;
  if (producer) {
    for (int i = 0; i < kImgMaxBufs; ++i) {
      mbar_init(full + 8u * i, 1);
      mbar_init(empty + 8u * i, kImgWarps);
    }
    mbar_init(cbar, kImgWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // the first copies start before the rest of the block has set up: every buffer is free
    for (; q < total && q < P.nbuf; ++q) issue_chunk();
  }
  // bytes of channels beyond C (C % 32 != 0) are never written by a unit: they stay zero
  for (int i = tid; i < nplanes * HW * P.Cw; i += kImgThreads) reinterpret_cast<uint32_t *>(wbytes)[i] = 0u;
  if (kHasBN)
    for (int c = tid; c < P.C; c += kImgThreads) bn[c] = make_float2(__ldg(P.scale + c), __ldg(P.shift + c));
  __syncthreads();

  if (warp == kImgWarps) {
    // ---- producer: one thread issues every copy of this block
    if (lane == 0) {
      bool ok = true;
      for (; q < total; ++q) {
        ok = mbar_wait(empty + 8u * pb, eph, abort_flag, &g_status_act);
        if (!ok) break;
        issue_chunk();
      }
      if (!ok) {
        // gave up: the copies already issued (at most one per buffer) must land before the
        // block's shared memory is released
        for (long long back = 1; back <= P.nbuf && back <= q; ++back) {
          const long long c = q - back;
          const uint32_t bar = full + 8u * (uint32_t)(c % P.nbuf), par = (uint32_t)(c / P.nbuf) & 1u;
          for (int i = 0; i < (1 << 20) && !mbar_try(bar, par); ++i) {}
        }
      }
    }
    return;
  }

  // ---- consumers
  // Warp -> (pixel groups, 8-channel blocks): with at least eight pixel groups a warp takes the
  // groups warp, warp + 8, ... (at most kImgRounds) and every channel block; with fewer, the
  // warps of a pixel group share the channel blocks (slot, slot + slots, ...).
  const int slots = npg >= kImgWarps ? 1 : kImgWarps / npg;
  const int pg0 = npg >= kImgWarps ? warp : warp % npg;
  const int slot = npg >= kImgWarps ? 0 : warp / npg;
  const bool has_work = slot < slots;
  // k <= 2: tau_1 .. tau_3 (k = 1 has tau_1 = 0 alone: the other two never compare true)
  const float kInf = __int_as_float(0x7f800000);
  const float t1 = kKbit ? tau[1] : 0.0f;
  const float t2 = kKbit && P.kbits == 2 ? tau[2] : kInf, t3 = kKbit && P.kbits == 2 ? tau[3] : kInf;
  const int pstep = 32 * kImgWarps;
  const uint32_t plane4 = (uint32_t)HW * 4u;
  const uint32_t bn_addr = base + P.off_bn;
  int b = 0;
  uint32_t fph = 0u, cph = 0u;
  for (int n = blockIdx.x; n < P.N; n += gridDim.x) {
    float asum[kImgRounds];
#pragma unroll
    for (int r = 0; r < kImgRounds; ++r) asum[r] = 0.0f;
    for (int ch = 0; ch < nchunks; ++ch) {
      if (!mbar_wait(full + 8u * b, fph, abort_flag, &g_status_act)) return;
      if (has_work) {
        // 32-bit shared addresses: one add per load (the stride between channels is H W words)
        const uint32_t buf = base + P.off_buf + (uint32_t)b * P.chunk_bytes + (uint32_t)(pg0 * 32 + lane) * 4u;
        for (int sb = slot; sb < nsub; sb += slots) {
          const int c0 = ch * P.cc + sb * 8;
          float4 ss[4];                       // (scale, shift) of two channels per load
          if (kHasBN) {
#pragma unroll
            for (int j = 0; j < 4; ++j) ss[j] = lds_f4(bn_addr + (uint32_t)(c0 + 2 * j) * 8u);
          }
          uint32_t ta[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) ta[j] = buf + (uint32_t)(sb * 8 + j) * plane4;
          uint8_t *wb = wbytes + (size_t)(pg0 * 32 + lane) * (P.Cw * 4) + (c0 >> 3);
#pragma unroll
          for (int r = 0; r < kImgRounds; ++r) {
            if (pg0 * 32 + lane + r * pstep < HW) {
              float y[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) y[j] = lds_f(ta[j] + (uint32_t)(r * pstep * 4));
              uint32_t bits = 0u;              // sign mode: the 8 bits; k-bit: plane p in byte p (k <= 4)
              uint32_t bits_hi = 0u;           // planes 4 .. 6
              float p0 = 0.0f, p1 = 0.0f;
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float v = y[j];
                if (kHasBN) v = (j & 1) ? __fmaf_rn(ss[j >> 1].z, v, ss[j >> 1].w) : __fmaf_rn(ss[j >> 1].x, v, ss[j >> 1].y);
                if (kKbit) {
                  // largest index whose decision point is <= v, by bisection over the sorted tau
                  int idx = 0;
                  if (P.kbits <= 2) {           // up to three decision points, held in registers
                    idx = (v >= t1 ? 1 : 0) + (v >= t2 ? 1 : 0) + (v >= t3 ? 1 : 0);
                  } else {
                    for (int bb = P.kbits - 1; bb >= 0; --bb) {
                      const int cand = idx + (1 << bb);
                      if (v >= tau[cand]) idx = cand;
                    }
                  }
                  // bit p of idx -> bit j of byte p: spread the low four bits over four bytes
                  const uint32_t lo = (uint32_t)idx & 15u, hi = (uint32_t)idx >> 4;
                  if (P.kbits <= 2) {
                    bits |= ((lo & 1u) | ((lo & 2u) << 7)) << j;
                  } else {
                    bits |= ((lo & 1u) | ((lo & 2u) << 7) | ((lo & 4u) << 14) | ((lo & 8u) << 21)) << j;
                    if (P.kbits > 4) bits_hi |= ((hi & 1u) | ((hi & 2u) << 7) | ((hi & 4u) << 14)) << j;
                  }
                } else {
                  if (v >= 0.0f) bits |= 1u << j;
                }
                if (j & 1) p1 += fabsf(v); else p0 += fabsf(v);
              }
              if (kKbit) {
                for (int pl = 0; pl < P.kbits; ++pl)
                  wb[(size_t)pl * plane_bytes + (size_t)(r * pstep) * (P.Cw * 4)] =
                      (uint8_t)((pl < 4 ? bits >> (8 * pl) : bits_hi >> (8 * (pl - 4))) & 0xFFu);
              } else {
                wb[(size_t)(r * pstep) * (P.Cw * 4)] = (uint8_t)bits;
              }
              asum[r] += p0 + p1;
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty + 8u * b);
      if (++b == P.nbuf) { b = 0; fph ^= 1u; }
    }
    if (has_work) {
#pragma unroll
      for (int r = 0; r < kImgRounds; ++r)
        if (pg0 * 32 + lane + r * pstep < HW) apart[slot * HW + pg0 * 32 + lane + r * pstep] = asum[r];
    }
    // the image is packed: A, the packed words, then K from the A just formed
    if (!img_sync(cbar, cph, lane, abort_flag)) return;
    for (int p = tid; p < HW; p += 32 * kImgWarps) {
      float sum = 0.0f;
      for (int s = 0; s < slots; ++s) sum += apart[s * HW + p];
      const float a = sum / (float)P.C;
      P.A[(size_t)n * HW + p] = a;
      aimg[p] = a;
    }
    for (int pl = 0; pl < nplanes; ++pl) {
      uint32_t *dst = P.x_packed + ((size_t)pl * P.N + n) * HW * P.Cw;
      const uint32_t *srcw = reinterpret_cast<const uint32_t *>(wbytes + (size_t)pl * plane_bytes);
      for (int i = tid; i < HW * P.Cw; i += 32 * kImgWarps) dst[i] = srcw[i];
    }
    if (!img_sync(cbar, cph, lane, abort_flag)) return;
    const int HoWo = P.Ho * P.Wo;
    for (int i = tid; i < HoWo; i += 32 * kImgWarps) {
      const int oy = i / P.Wo, ox = i - oy * P.Wo;
      const int y0 = oy * P.stride - P.pad, x0 = ox * P.stride - P.pad;
      float s = 0.0f;
      if (KS > 0) {
        // square KS x KS filter: every tap a predicated load in straight-line code, summed in
        // tap order (taps outside the image add zero)
        float v[KS > 0 ? KS * KS : 1];
#pragma unroll
        for (int ky = 0; ky < KS; ++ky)
#pragma unroll
          for (int kx = 0; kx < KS; ++kx) {
            const int iy = y0 + ky, ix = x0 + kx;
            const bool in = iy >= 0 && iy < P.H && ix >= 0 && ix < P.W;
            v[ky * KS + kx] = in ? aimg[iy * P.W + ix] : 0.0f;
          }
#pragma unroll
        for (int t = 0; t < KS * KS; ++t) s += v[t];
      } else {
        const int ky0 = y0 < 0 ? -y0 : 0, ky1 = min(P.kh, P.H - y0);
        const int kx0 = x0 < 0 ? -x0 : 0, kx1 = min(P.kw, P.W - x0);
        for (int ky = ky0; ky < ky1; ++ky) {
          const float *row = aimg + (y0 + ky) * P.W + x0;
          for (int kx = kx0; kx < kx1; ++kx) s += row[kx];
        }
      }
      int div = P.kh * P.kw;
      if (P.valid_taps) {
        const int ny = min(P.kh, P.H - y0) - max(0, -y0), nx = min(P.kw, P.W - x0) - max(0, -x0);
        div = (ny > 0 && nx > 0) ? ny * nx : 0;
      }
      P.K[(size_t)n * HoWo + i] = div > 0 ? s / (float)div : 0.0f;
    }
  }
}

// K = box filter of zero-padded A.  One thread per output; blockIdx.y = image, so the index
// arithmetic is 32-bit and cheap.  KS > 0: square KS x KS filter, every tap a predicated load
// in straight-line code, so all of a thread's loads are in flight together (a loop with
// run-time bounds issues them one L2 round trip at a time).  KS = 0: any size.
template <int KS>
__global__ void __launch_bounds__(256)
box_filter_kernel(const float *__restrict__ A, int H, int W, int kh, int kw, int stride, int pad,
                  int Ho, int Wo, int valid_taps, float *__restrict__ K) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= Ho * Wo) return;
  const int oy = i / Wo, ox = i - oy * Wo;
  const float *a = A + (size_t)blockIdx.y * H * W;
  const int y0 = oy * stride - pad, x0 = ox * stride - pad;
  float s = 0.0f;
  if (KS > 0) {
    float v[KS > 0 ? KS * KS : 1];
#pragma unroll
    for (int ky = 0; ky < KS; ++ky)
#pragma unroll
      for (int kx = 0; kx < KS; ++kx) {
        const int iy = y0 + ky, ix = x0 + kx;
        const bool in = iy >= 0 && iy < H && ix >= 0 && ix < W;
        v[ky * KS + kx] = in ? __ldg(a + iy * W + ix) : 0.0f;
      }
#pragma unroll
    for (int t = 0; t < KS * KS; ++t) s += v[t];
  } else {
    const int ky0 = y0 < 0 ? -y0 : 0, ky1 = min(kh, H - y0);
    const int kx0 = x0 < 0 ? -x0 : 0, kx1 = min(kw, W - x0);
    for (int ky = ky0; ky < ky1; ++ky) {
      const float *row = a + (y0 + ky) * W + x0;
      for (int kx = kx0; kx < kx1; ++kx) s += __ldg(row + kx);
    }
  }
  // divisor: k_h k_w (zero-padded A), or the number of taps inside the image
  int div = kh * kw;
  if (valid_taps) {
    const int ny = min(kh, H - y0) - max(0, -y0), nx = min(kw, W - x0) - max(0, -x0);
    div = (ny > 0 && nx > 0) ? ny * nx : 0;
  }
  K[(size_t)blockIdx.y * Ho * Wo + i] = div > 0 ? s / (float)div : 0.0f;
}

}  // namespace

cudaError_t launch_box_filter(const float *A, const ConvGeom &g, float *K, cudaStream_t st);

namespace {

constexpr size_t kPackSmemMax = 100 * 1024;      // three blocks per SM

struct PackPlan { int G, PG; size_t smem; };

size_t pack_smem(int Cw, bool bn, int G, int PG) {
  return (size_t)kWarps * kBufsPerWarp * kTileFloats * sizeof(float) +
         (bn ? (size_t)Cw * 32 * sizeof(float2) : 0) + (size_t)PG * kPix * Cw * sizeof(uint32_t) +
         (size_t)PG * G * kPix * sizeof(float);
}

// With enough pixel groups to fill the GPU every warp packs whole pixel groups on its own
// (G = 1); otherwise, or when the staged words of eight pixel groups do not fit shared
// memory (many channels), the channel words of a pixel group are spread over the warps.
bool pack_plan(const ConvGeom &g, bool bn, PackPlan *pl) {
  const long long total_pix = (long long)g.N * g.H * g.W;
  const long long ngroups = (total_pix + kPix - 1) / kPix;
  const int Gs = g.Cw < kWarps ? g.Cw : kWarps;
  int G = ngroups >= 2048 ? 1 : Gs;
  if (pack_smem(g.Cw, bn, G, kWarps / G) > kPackSmemMax) G = Gs;
  pl->G = G;
  pl->PG = kWarps / G;
  pl->smem = pack_smem(g.Cw, bn, G, pl->PG);
  return pl->smem <= kPackSmemMax;
}

constexpr size_t kImgSmemMax = 112 * 1024;       // two blocks per SM
constexpr uint32_t kImgHeader = 256;             // barriers and the abort flag

// Whether the whole-image kernel serves this call, and with which chunking: planes that are
// not a multiple of four pixels, whole bytes of packed channels (with the 16-byte alignment of
// x that the entry point checks, every image then starts on a 16-byte boundary), enough images to occupy the SMs, and a chunk of at least eight channel planes
// small enough that two (better four) of them fit beside the staged outputs of an image.
bool image_plan(const ConvGeom &g, bool bn, int sms, int kbits, ImgParams *ip) {
  const long long HW = (long long)g.H * g.W;
  if ((HW & 3) == 0 || (g.C & 7) != 0) return false;
  if (g.N < sms / 2 || HW > 32 * kImgWarps * kImgRounds) return false;
  const int npg = (int)((HW + 31) / 32);
  const int slots = npg >= kImgWarps ? 1 : kImgWarps / npg;
  for (int pass = 0; pass < 3; ++pass) {
    const int nbuf = pass == 0 ? 4 : pass == 1 ? 3 : 2;
    const long long chunk_max = pass == 0 ? 24 * 1024 : pass == 1 ? 32 * 1024 : 48 * 1024;
    // the largest chunk of whole channel planes (a multiple of 8 that divides C) under the
    // pass's chunk size that fits shared memory beside the staged outputs of an image
    for (int cc = g.C; cc >= 8; cc -= 8) {
      if (g.C % cc != 0 || (long long)cc * HW * 4 > chunk_max) continue;
      const uint32_t chunk = (uint32_t)(cc * HW * 4);
      uint32_t off = kImgHeader;
      ip->off_buf = off; off += (uint32_t)nbuf * chunk;
      ip->off_words = off; off += (uint32_t)((kbits > 0 ? kbits : 1) * HW * g.Cw * 4);
      ip->off_apart = off; off += (uint32_t)(slots * HW * 4);
      ip->off_aimg = off; off += (uint32_t)(HW * 4);
      off = (off + 15u) & ~15u;
      ip->off_bn = off; off += bn ? (uint32_t)g.C * 8u : 0u;
      if (off > kImgSmemMax) continue;
      ip->cc = cc; ip->nbuf = nbuf; ip->chunk_bytes = chunk; ip->kbits = kbits;
      return true;
    }
  }
  return false;
}

template <bool kHasBN, int KS, bool kKbit>
cudaError_t launch_image_variant(const ImgParams &ip, int sms, size_t smem, cudaStream_t st) {
  static bool attr_flags[64] = {};
  bool &attr_set = attr_done_for_current_device(attr_flags);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(binactiv_image_kernel<kHasBN, KS, kKbit>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kImgSmemMax);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, binactiv_image_kernel<kHasBN, KS, kKbit>, kImgThreads,
                                                    smem) != cudaSuccess || per_sm < 1) {
    (void)cudaGetLastError();
    per_sm = 1;
  }
  const long long resident = (long long)per_sm * sms;
  const unsigned grid = (unsigned)(ip.N < resident ? ip.N : resident);
  binactiv_image_kernel<kHasBN, KS, kKbit><<<grid, kImgThreads, smem, st>>>(ip);
  return cudaGetLastError();
}

void fill_img_params(ImgParams &ip, const float *x, const float *scale, const float *shift,
                     const ConvGeom &g, uint32_t *x_packed, float *A, float *K) {
  ip.x = x; ip.scale = scale; ip.shift = shift; ip.x_packed = x_packed; ip.A = A; ip.K = K;
  ip.N = g.N; ip.C = g.C; ip.H = g.H; ip.W = g.W; ip.Cw = g.Cw;
  ip.kh = g.kh; ip.kw = g.kw; ip.stride = g.stride; ip.pad = g.pad; ip.Ho = g.Ho; ip.Wo = g.Wo;
  ip.valid_taps = (g.flags & XNOR_FLAG_K_VALID_TAPS) ? 1 : 0;
}

cudaError_t launch_binactiv_image(const ImgParams &ip, bool bn, int sms, cudaStream_t st) {
  const size_t smem = (size_t)ip.off_bn + (bn ? (size_t)ip.C * 8 : 0);
  const int ks = ip.kh == ip.kw ? ip.kh : 0;
#define XNOR_IMG(KS) (ip.kbits > 0 ? (bn ? launch_image_variant<true, KS, true>(ip, sms, smem, st)    \
                                       : launch_image_variant<false, KS, true>(ip, sms, smem, st))  \
                                  : (bn ? launch_image_variant<true, KS, false>(ip, sms, smem, st)   \
                                       : launch_image_variant<false, KS, false>(ip, sms, smem, st)))
  if (ks == 1) return XNOR_IMG(1);
  if (ks == 3) return XNOR_IMG(3);
  if (ks == 5) return XNOR_IMG(5);
  if (ks == 7) return XNOR_IMG(7);
  return XNOR_IMG(0);
#undef XNOR_IMG
}

}  // namespace

int binactiv_kbit_launch_count(const ConvGeom &g, bool has_bn, int kbits) {
  ImgParams ip;
  return image_plan(g, has_bn, sm_count_of_current_device(), kbits, &ip) ? 1 : 2;
}

int binactiv_launch_count(const ConvGeom &g, bool has_bn) { return binactiv_kbit_launch_count(g, has_bn, 0); }

cudaError_t read_status_act(int *status) {
  cudaError_t e = cudaMemcpyFromSymbol(status, g_status_act, sizeof(int));
  if (e == cudaSuccess && *status != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_status_act, &zero, sizeof(int));
  }
  return e;
}

// Shapes the BinActiv kernels cover: the staged words fit shared memory (C_in <= 2976 with a
// BatchNorm affine, more without) and one grid row per image.
bool binactiv_supported(const ConvGeom &g, bool has_bn) {
  PackPlan pl;
  return g.N <= 65535 && pack_plan(g, has_bn, &pl);
}

cudaError_t launch_binactiv(const float *x, const float *scale, const float *shift,
                            const ConvGeom &g, uint32_t *x_packed, float *A, float *K,
                            cudaStream_t st) {
  const long long total_pix = (long long)g.N * g.H * g.W;
  PackPlan pl;
  if (g.N > 65535 || !pack_plan(g, scale != nullptr, &pl)) return cudaErrorInvalidValue;
  const int sms = sm_count_of_current_device();
  {
    ImgParams ip;
    if (image_plan(g, scale != nullptr, sms, 0, &ip)) {
      fill_img_params(ip, x, scale, shift, g, x_packed, A, K);
      return launch_binactiv_image(ip, scale != nullptr, sms, st);
    }
  }
  const int G = pl.G, PG = pl.PG;
  const size_t smem = pl.smem;
  static bool attr_flags[64] = {};
  bool &attr_set = attr_done_for_current_device(attr_flags);
  if (!attr_set) {
    cudaError_t e = cudaSuccess;
    const void *kernels[4] = {(const void *)binactiv_pack_kernel<true, true>,
                              (const void *)binactiv_pack_kernel<true, false>,
                              (const void *)binactiv_pack_kernel<false, true>,
                              (const void *)binactiv_pack_kernel<false, false>};
    for (int i = 0; i < 4 && e == cudaSuccess; ++i)
      e = cudaFuncSetAttribute(kernels[i], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPackSmemMax);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  const long long nbatches = ((total_pix + kPix - 1) / kPix + PG - 1) / PG;
  const bool v16 = ((g.H * g.W) & 3) == 0;
  // persistent grid: as many blocks as are resident at once (the shared-memory split the driver
  // picks for this kernel decides whether two or three fit an SM), so that no block waits for
  // a second wave
  const void *kern = scale ? (v16 ? (const void *)binactiv_pack_kernel<true, true>
                                  : (const void *)binactiv_pack_kernel<true, false>)
                           : (v16 ? (const void *)binactiv_pack_kernel<false, true>
                                  : (const void *)binactiv_pack_kernel<false, false>);
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 32 * kWarps, smem) != cudaSuccess ||
      per_sm < 1) {
    (void)cudaGetLastError();
    per_sm = 2;
  }
  const long long resident = (long long)per_sm * sms;
  const unsigned grid = (unsigned)(nbatches < resident ? nbatches : resident);
#define XNOR_PACK(BN, V16) binactiv_pack_kernel<BN, V16><<<grid, 32 * kWarps, smem, st>>>( \
      x, scale, shift, total_pix, g.C, g.H * g.W, g.Cw, G, PG, x_packed, A)
  if (scale) { if (v16) XNOR_PACK(true, true); else XNOR_PACK(true, false); }
  else { if (v16) XNOR_PACK(false, true); else XNOR_PACK(false, false); }
#undef XNOR_PACK
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_box_filter(A, g, K, st);
}

cudaError_t launch_box_filter(const float *A, const ConvGeom &g, float *K, cudaStream_t st) {
  if (g.N > 65535) return cudaErrorInvalidValue;
  const dim3 kgrid((unsigned)((g.Ho * g.Wo + 255) / 256), (unsigned)g.N);
  const int ks = g.kh == g.kw ? g.kh : 0;
  const int valid = (g.flags & XNOR_FLAG_K_VALID_TAPS) ? 1 : 0;
#define XNOR_BOX(KS) box_filter_kernel<KS><<<kgrid, 256, 0, st>>>(A, g.H, g.W, g.kh, g.kw, g.stride, \
                                                                g.pad, g.Ho, g.Wo, valid, K)
  if (ks == 1) XNOR_BOX(1);
  else if (ks == 3) XNOR_BOX(3);
  else if (ks == 5) XNOR_BOX(5);
  else if (ks == 7) XNOR_BOX(7);
  else XNOR_BOX(0);
#undef XNOR_BOX
  return cudaGetLastError();
}


namespace {

// A[i] = (part 0 + part 1 + ...)[i] / C, the parts added in index order.
__global__ void __launch_bounds__(256)
sum_parts_kernel(const float *__restrict__ parts, int nparts, size_t n, float C, float *__restrict__ A) {
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (size_t)gridDim.x * 256) {
    float s = 0.0f;
    for (int p = 0; p < nparts; ++p) s += __ldg(parts + (size_t)p * n + i);
    A[i] = s / C;
  }
}

}  // namespace

cudaError_t launch_binactiv_finish(const float *A_part, int parts, const ConvGeom &g, float *A,
                                   float *K, cudaStream_t st) {
  const size_t n = (size_t)g.N * g.H * g.W;
  const unsigned grid = (unsigned)std::min<size_t>((n + 255) / 256, (size_t)sm_count_of_current_device() * 8);
  sum_parts_kernel<<<grid, 256, 0, st>>>(A_part, parts, n, (float)g.C, A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_box_filter(A, g, K, st);
}

// ---------------------------------------------------------------------------
// BinActiv with k-bit activations (Section 3.2, "k-bit Quantization"):
//   q_k(x) = 2([(2^k - 1)(x + 1)/2]/(2^k - 1) - 1/2),  x in [-1, 1]
// replaces sign().  With i = [.] in 0 .. 2^k - 1 the level is (2i - (2^k-1))/(2^k-1); the
// kernel stores the index i as k bit planes (plane p, bit c % 32 of word c / 32 = bit p of i),
// so that the level code is sum_p 2^p (2 b_p - 1): a weighted sum of k ordinary +-1 planes.
// Values outside [-1, 1] are clipped; ties round up (k = 1 is then sign() with +1 at zero).
// The rounding decision is a comparison in fp32: i >= j exactly when
// y >= tau_j = fp32((2j - 1)/(2^k - 1) - 1).  A (and K) are those of the 1-bit block.
namespace {

__global__ void __launch_bounds__(256)
binactiv_pack_kbit_kernel(const float *__restrict__ x, const float *__restrict__ scale,
                          const float *__restrict__ shift, long long total_pix, int C, int HW, int Cw,
                          int kbits, uint32_t *__restrict__ x_planes, float *__restrict__ A) {
  __shared__ float tau[128];                 // tau[j], j = 1 .. 2^k - 1; tau[0] unused
  const int levels = (1 << kbits) - 1;
  for (int j = 1 + threadIdx.x; j <= levels; j += blockDim.x)
    tau[j] = (float)((double)(2 * j - 1) / (double)levels - 1.0);
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const long long ngroups = (total_pix + 31) / 32;
  const long long warp0 = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long grp = warp0; grp < ngroups; grp += nwarps) {
    const long long gp = grp * 32 + lane;          // this lane's pixel
    if (gp >= total_pix) continue;
    const long long n = gp / HW;
    const int p = (int)(gp - n * HW);
    const float *src = x + (size_t)n * C * HW + p;
    float asum = 0.0f;
    for (int cw = 0; cw < Cw; ++cw) {
      uint32_t words[7] = {0u, 0u, 0u, 0u, 0u, 0u, 0u};
      float p0 = 0.0f, p1 = 0.0f;
      const int c0 = cw * 32, nc = min(32, C - c0);
      for (int j0 = 0; j0 < nc; j0 += 8) {
        float yv[8];                       // eight loads in flight before any is used
#pragma unroll
        for (int q = 0; q < 8; ++q)
          yv[q] = j0 + q < nc ? __ldg(src + (size_t)(c0 + j0 + q) * HW) : 0.0f;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int j = j0 + q;
          if (j < nc) {
            float y = yv[q];
            if (scale != nullptr) y = __fmaf_rn(__ldg(scale + c0 + j), y, __ldg(shift + c0 + j));
            if (q & 1) p1 += fabsf(y); else p0 += fabsf(y);
            // largest index whose decision point is <= y, by bisection over the sorted tau
            int idx = 0;
            for (int b = kbits - 1; b >= 0; --b) {
              const int cand = idx + (1 << b);
              if (y >= tau[cand]) idx = cand;
            }
#pragma unroll
            for (int b = 0; b < 7; ++b)
              if (b < kbits) words[b] |= (uint32_t)((idx >> b) & 1) << j;
          }
        }
      }
      asum += p0 + p1;
#pragma unroll
      for (int b = 0; b < 7; ++b)
        if (b < kbits) x_planes[((size_t)b * total_pix + gp) * Cw + cw] = words[b];
    }
    A[gp] = asum / (float)C;
  }
}

}  // namespace

cudaError_t launch_binactiv_kbit(const float *x, const float *scale, const float *shift,
                                 const ConvGeom &g, int kbits, uint32_t *x_planes, float *A, float *K,
                                 cudaStream_t st) {
  {
    // planes of odd size and enough images: the kernel that streams whole images, in k-bit mode
    const int sms = sm_count_of_current_device();
    ImgParams ip;
    if (image_plan(g, scale != nullptr, sms, kbits, &ip)) {
      fill_img_params(ip, x, scale, shift, g, x_planes, A, K);
      return launch_binactiv_image(ip, scale != nullptr, sms, st);
    }
  }
  const long long total_pix = (long long)g.N * g.H * g.W;
  const long long nblocks = ((total_pix + 31) / 32 + 7) / 8;
  const unsigned grid = (unsigned)std::min<long long>(nblocks, 8ll * sm_count_of_current_device());
  binactiv_pack_kbit_kernel<<<grid, 256, 0, st>>>(x, scale, shift, total_pix, g.C, g.H * g.W, g.Cw,
                                                  kbits, x_planes, A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_box_filter(A, g, K, st);
}

// ---------------------------------------------------------------------------
// xnor_binactiv_static: the same two kernels, with the A plane kept in a
// fixed array of this library instead of a caller buffer.
namespace {

constexpr size_t kStaticPixels = XNOR_BINACTIV_STATIC_MAX_PIXELS;
constexpr int kMaxDevices = 64;

// Lives in the device memory of every GPU that loads the library, until exit.
static __device__ __align__(256) float g_static_A[kStaticPixels];

// In host code `g_static_A` is only a handle for the runtime; the device
// address has to be asked for, per device, with that device current.
float *g_static_A_ptr[kMaxDevices] = {};

cudaError_t static_A_address(float **ptr) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_static_A_ptr[dev] == nullptr) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_A);
    if (e != cudaSuccess) return e;
    g_static_A_ptr[dev] = static_cast<float *>(p);
  }
  *ptr = g_static_A_ptr[dev];
  return cudaSuccess;
}

}  // namespace

size_t binactiv_static_max_pixels() { return kStaticPixels; }

cudaError_t launch_binactiv_static(const float *x, const float *scale, const float *shift,
                                   const ConvGeom &g, uint32_t *x_packed, float *K,
                                   cudaStream_t st) {
  float *A = nullptr;
  cudaError_t e = static_A_address(&A);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
  // every A value the box filter reads is written by the pack kernel of this call first,
  // so nothing left by an earlier call is ever used and nothing needs clearing
  return launch_binactiv(x, scale, shift, g, x_packed, A, K, st);
}

}  // namespace xnor
