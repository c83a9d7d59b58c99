// BinConv on the 5th-generation tensor cores (Eq. 11): persistent,
// warp-specialised implicit GEMM on tcgen05.mma kind::mxf4.
//
// sign(I) (*) sign(W) is an exact integer contraction.  Both operands become
// e2m1 (4-bit) numbers whose products are all +-1, block scales are 1, and the
// fp32 accumulators in tensor memory hold exact integers (|sum| < 2^24).  HBM
// only ever sees the 1-bit packed words; a CTA expands what it needs into
// shared memory.
//
//  GEMM roles.  D[pixel][filter] = sum_k X[pixel][k] * Wt[filter][k]:
//    A (M = 128 rows) = 128 consecutive positions of a virtual pixel stream.
//        For stride s the input is split into s*s phase planes (plane (py,px)
//        holds input pixels (s*r+py, s*c+px)); every plane is laid out as one
//        long stream in which each row is preceded by `lead` zero pixels and
//        each image by `leadY` zero rows.  With GEMM row m = stream index of
//        an output pixel, filter tap (ky,kx) reads, in ONE phase plane, stream
//        position m + shift(ky,kx): a pure shift.  So the pixels a tile
//        touches are expanded ONCE into the no-swizzle K-major operand layout
//        (8 pixels x 16 bytes per core matrix, pixels contiguous, one plane
//        per 32 channels) and every tap's A operand is that patch at a shifted
//        start address.  Zero pixels and the channel tail expand to the value
//        0, so padded taps contribute exactly 0 with no mask or correction.
//        Stream positions that are padding give junk rows that are never stored.
//    B (N = NT rows)  = a slab of NT filters, expanded from bits by producer
//        warps into a ring of shared-memory stages, in the order of a table of
//        K-steps (one MMA of K = 64 = two 32-channel pieces each) that every
//        CTA builds once.  A piece is (tap, channel word); when the number of
//        channel words is odd the last word of two consecutive taps shares an
//        MMA, so no K-step is wasted on padding.
//
//  Encodings.  A packed word holds 32 sign bits; it becomes 32 e2m1 nibbles in
//  four registers, register r holding channels r, r+4, ..., r+28.  Activations
//  are +-{2, 1, 0.5, 0.5} for r = 0..3, weights +-{0.5, 1, 2, 2}: every product
//  is the product of the two signs.
//
//  Roles (480 threads, one CTA per SM, CTAs loop over work items = (pixel
//  tile, filter slab)): warps 0-7 epilogue (tensor memory -> registers ->
//  coalesced NCHW stores of D * K * alpha (+ residual)), warp 8 issues the
//  MMAs, warps 9-12 expand weights, warps 13-14 expand activation patches.
//  Accumulators are double-buffered in tensor memory so the epilogue of one
//  item overlaps the MMAs of the next.  Every wait is bounded: on expiry the
//  CTA records XNOR_ERR_TIMEOUT in a device status word, stops, frees its
//  tensor memory and exits.
#include <algorithm>

#include "common.cuh"
#include "umma_common.cuh"

namespace xnor {

__device__ int g_status_tc = 0;

namespace {

using namespace umma;

constexpr int kEpiWarps = 8;
constexpr int kMmaWarp = 8;
constexpr int kWgtWarp0 = 9, kWgtWarps = 4, kWgtThreads = 32 * kWgtWarps;
constexpr int kPatWarp0 = 13, kPatWarps = 2, kPatThreads = 32 * kPatWarps;
constexpr int kThreads = 32 * (kPatWarp0 + kPatWarps);     // 480
constexpr int kTileM = 128;          // stream positions per tile = tensor-memory lanes
constexpr int kTmemCols = 512;
constexpr int kSfCol = 480;          // columns [480, 512): unit block scales
constexpr int kMaxAccCols = 480;
constexpr int kMaxStages = 6;
constexpr int kMaxPatchBufs = 4;
constexpr int kMaxSteps = 1024;      // K-steps (MMAs) per work item
constexpr int kPrefetch = 3;         // weight stages whose packed words are in flight
constexpr int kUnits = 4;            // (row, K-step) units per weight thread per stage
constexpr size_t kCtrlBytes = 512;
constexpr size_t kSmemMax = 232448 - 1024;

struct TcParams {
  const uint32_t *xp, *wp;
  const float *alpha, *K, *residual;
  float *out;
  int32_t *acc_out;
  int N, C, H, W, Co, kh, kw, stride, pad, Ho, Wo, Cw;
  int Hq, Wq, leadY, leadX;    // stream geometry of every phase plane
  int dymin, dxmin;
  long long L;                 // stream length N*Hq*Wq
  int ntiles, nslabs, NT;      // pixel tiles, filter slabs, filters per slab (multiple of 16)
  int nacc;                    // accumulator buffers in tensor memory (1 or 2)
  int ppix;                    // stream positions staged per phase plane (128 + halo, rounded to 8)
  int nplanes;                 // stride*stride*Cw operand planes per patch
  int npb;                     // patch buffers
  int nsteps;                  // K-steps per item
  int mps;                     // K-steps per weight stage
  int stages;
  int rows_mod, grp_steps;     // weight-thread mapping (see weight producer)
  uint32_t patch_bytes, stage_bytes;
  uint32_t off_table, off_ring, off_patch;   // byte offsets in dynamic shared memory
  uint32_t idesc;
  uint32_t tail_mask;          // bits of real channels in the last word
};

// One K-step: A-operand start offset inside a patch, distance between its two
// 32-channel pieces, and the two packed words of a filter row it consumes
// (index within the row's [tap][Cw] words; 0xFFFFFFFF = no second piece).
struct __align__(16) KStep {
  uint32_t a_off, a_lbo, gw1, gw2;
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

// 32 sign bits -> 32 e2m1 nibbles (sign in bit 3 of a nibble, magnitude code
// 1 = 0.5, 2 = 1, 4 = 2).  Register r holds channels r, r+4, ...; a set bit is +.
// kAct: magnitudes {2, 1, 0.5, 0.5}; otherwise {0.5, 1, 2, 2}.
template <bool kAct>
__device__ __forceinline__ void expand_signs(uint32_t w, uint32_t v[4]) {
  constexpr uint32_t m0 = kAct ? 0xCCCCCCCCu : 0x99999999u;
  constexpr uint32_t m1 = 0xAAAAAAAAu;
  constexpr uint32_t m2 = kAct ? 0x99999999u : 0xCCCCCCCCu;
  constexpr uint32_t m3 = kAct ? 0x99999999u : 0xCCCCCCCCu;
  v[0] = ((w << 3) & 0x88888888u) ^ m0;
  v[1] = ((w << 2) & 0x88888888u) ^ m1;
  v[2] = ((w << 1) & 0x88888888u) ^ m2;
  v[3] = (w & 0x88888888u) ^ m3;
}

// Shift of a filter tap inside a phase plane, and the plane it reads.
__device__ __forceinline__ void tap_geometry(const TcParams &P, int tap, int &phase, int &shift) {
  const int ky = tap / P.kw, kx = tap - ky * P.kw;
  const int ay = ky - P.pad, ax = kx - P.pad;
  // floor division / non-negative remainder by the stride
  const int dy = (ay >= 0) ? ay / P.stride : -((-ay + P.stride - 1) / P.stride);
  const int dx = (ax >= 0) ? ax / P.stride : -((-ax + P.stride - 1) / P.stride);
  const int py = ay - dy * P.stride, px = ax - dx * P.stride;
  phase = py * P.stride + px;
  shift = (dy - P.dymin) * P.Wq + (dx - P.dxmin);
}

// Piece (tap, w) -> byte offset of its A operand inside a patch.
__device__ __forceinline__ uint32_t piece_offset(const TcParams &P, int tap, int w) {
  int phase, shift;
  tap_geometry(P, tap, phase, shift);
  return (uint32_t)(phase * P.Cw + w) * ((uint32_t)P.ppix * 16u) + (uint32_t)shift * 16u;
}

// K-step j of the fixed order: for every pair of taps (t, t+1): the word pairs
// of t, the word pairs of t+1, then (Cw odd only) the last words of t and t+1
// together.  A lone last tap pairs its last word with nothing.
__device__ void build_kstep(const TcParams &P, int j, KStep &ks) {
  const int taps = P.kh * P.kw, Cw = P.Cw, h = Cw >> 1;
  int t1, w1, t2, w2;
  if ((Cw & 1) == 0) {
    t1 = j / h; w1 = 2 * (j - t1 * h); t2 = t1; w2 = w1 + 1;
  } else {
    const int per_pair = 2 * h + 1;
    const int pp = j / per_pair, rem = j - pp * per_pair;
    const int ta = 2 * pp;
    const bool lone = ta + 1 >= taps;          // last tap without a partner
    if (rem < h) { t1 = ta; w1 = 2 * rem; t2 = t1; w2 = w1 + 1; }
    else if (!lone && rem < 2 * h) { t1 = ta + 1; w1 = 2 * (rem - h); t2 = t1; w2 = w1 + 1; }
    else { t1 = ta; w1 = Cw - 1; t2 = lone ? -1 : ta + 1; w2 = Cw - 1; }
  }
  ks.a_off = piece_offset(P, t1, w1);
  ks.gw1 = (uint32_t)(t1 * Cw + w1);
  if (t2 >= 0) {
    uint32_t o2 = piece_offset(P, t2, w2);
    ks.gw2 = (uint32_t)(t2 * Cw + w2);
    if (o2 < ks.a_off) {       // the piece at the lower address goes first
      const uint32_t o = ks.a_off, g = ks.gw1;
      ks.a_off = o2; ks.gw1 = ks.gw2; o2 = o; ks.gw2 = g;
    }
    ks.a_lbo = o2 - ks.a_off;
  } else {
    ks.a_lbo = 16u;            // any in-bounds piece: its weights are 0
    ks.gw2 = 0xFFFFFFFFu;
  }
}

struct Smem {
  uint32_t wfull, wempty, pfull, pempty, afull, aempty;   // shared-space addresses of barrier arrays
  uint32_t *tmem_slot;
  volatile int *abort_flag;
  const KStep *table;
  uint32_t ring, patch;                                   // shared-space byte addresses
};

__device__ __forceinline__ Smem carve(uint8_t *smem, const TcParams &P) {
  Smem s;
  const uint32_t base = smem_u32(smem);
  s.wfull = base;
  s.wempty = s.wfull + 8u * kMaxStages;
  s.pfull = s.wempty + 8u * kMaxStages;
  s.pempty = s.pfull + 8u * kMaxPatchBufs;
  s.afull = s.pempty + 8u * kMaxPatchBufs;
  s.aempty = s.afull + 16u;
  s.tmem_slot = reinterpret_cast<uint32_t *>(smem + 8 * (2 * kMaxStages + 2 * kMaxPatchBufs + 4));
  s.abort_flag = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
  s.table = reinterpret_cast<const KStep *>(smem + P.off_table);
  s.ring = base + P.off_ring;
  s.patch = base + P.off_patch;
  return s;
}

// ------------------------------------------------------------------ MMA issuer (one warp)
__device__ void mma_role(const TcParams &P, const Smem &S, long long i0, long long i1,
                         uint32_t tmem_base, int lane) {
  const uint32_t tmem_sf = tmem_base + (uint32_t)kSfCol;
  const int nst = (P.nsteps + P.mps - 1) / P.mps;
  const uint32_t b_lbo = (uint32_t)P.NT * 16u;
  int ws = 0, pb = 0;
  uint32_t wph = 0, pph = 0;
  long long k = 0;                       // items done by this CTA
  int tile = (int)(i0 / P.nslabs), slab = (int)(i0 - (long long)tile * P.nslabs);
  bool ok = true, new_tile = true;
  uint32_t patch_addr = 0;
  for (long long item = i0; item < i1 && ok; ++item, ++k) {
    if (new_tile) {
      ok = mbar_wait(S.pfull + 8u * pb, pph, S.abort_flag, &g_status_tc);
      if (!ok) break;
      patch_addr = S.patch + (uint32_t)pb * P.patch_bytes;
    }
    const int ab = (int)(k % P.nacc);
    const uint32_t use = (uint32_t)(k / P.nacc);
    ok = mbar_wait(S.aempty + 8u * ab, (use & 1u) ^ 1u, S.abort_flag, &g_status_tc);
    if (!ok) break;
    tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)(ab * P.NT);
    uint32_t accumulate = 0;
    for (int st = 0; st < nst && ok; ++st) {
      ok = mbar_wait(S.wfull + 8u * ws, wph, S.abort_flag, &g_status_tc);
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) {
        const int j0 = st * P.mps;
        const int nj = min(P.mps, P.nsteps - j0);
        uint32_t b_addr = S.ring + (uint32_t)ws * P.stage_bytes;
        for (int jj = 0; jj < nj; ++jj) {
          const KStep ks = S.table[j0 + jj];
          umma_mxf4(d_tmem, make_desc(patch_addr + ks.a_off, ks.a_lbo, 128u),
                    make_desc(b_addr, b_lbo, 128u), P.idesc, tmem_sf, tmem_sf, accumulate);
          accumulate = 1;
          b_addr += 2u * b_lbo;
        }
        umma_commit(S.wempty + 8u * ws);
      }
      __syncwarp();
      if (++ws == P.stages) { ws = 0; wph ^= 1u; }
    }
    if (!ok) break;
    // next item: same tile (next slab) or the next tile
    new_tile = false;
    if (++slab == P.nslabs) { slab = 0; ++tile; new_tile = true; }
    if (lane == 0) {
      umma_commit(S.afull + 8u * ab);
      if (new_tile || item + 1 == i1) umma_commit(S.pempty + 8u * pb);
    }
    __syncwarp();
    if (new_tile) { if (++pb == P.npb) { pb = 0; pph ^= 1u; } }
  }
}

// ------------------------------------------------------------------ weight producers (4 warps)
struct WCursor {
  long long item;
  int st, slab;
};

__device__ void weight_role(const TcParams &P, const Smem &S, long long i0, long long i1, int wt,
                            int lane) {
  const int nst = (P.nsteps + P.mps - 1) / P.mps;
  const int row0 = wt % P.rows_mod, grp = wt / P.rows_mod;
  const int gs = P.grp_steps;            // 1, 2 or 4
  const int gs_log = 31 - __clz(gs);
  const int nrows = P.NT > 128 ? 2 : 1;
  const size_t row_words = (size_t)P.kh * P.kw * P.Cw;
  const uint32_t b_lbo = (uint32_t)P.NT * 16u;
  const int slab0 = (int)(i0 % P.nslabs);
  WCursor fc{i0, 0, slab0}, cc{i0, 0, slab0};
  auto advance = [&](WCursor &c) {
    if (++c.st == nst) { c.st = 0; ++c.item; if (++c.slab == P.nslabs) c.slab = 0; }
  };
  uint32_t pf[kPrefetch][2 * kUnits];
  // unit u = rr * gs + kk: filter row row0 + 128 rr, K-step (st * mps + grp * gs + kk)
  auto fetch = [&](uint32_t dst[2 * kUnits], const WCursor &c) {
#pragma unroll
    for (int u = 0; u < kUnits; ++u) {
      dst[2 * u] = 0u; dst[2 * u + 1] = 0u;
      const int rr = u >> gs_log, kk = u & (gs - 1);
      const int row = row0 + 128 * rr;
      const int j = c.st * P.mps + grp * gs + kk;
      const int co = c.slab * P.NT + row;
      if (c.item < i1 && rr < nrows && row < P.NT && co < P.Co && j < P.nsteps) {
        const KStep ks = S.table[j];
        const uint32_t *rowp = P.wp + (size_t)co * row_words;
        dst[2 * u] = __ldg(rowp + ks.gw1);
        if (ks.gw2 != 0xFFFFFFFFu) dst[2 * u + 1] = __ldg(rowp + ks.gw2);
      }
    }
  };
#pragma unroll
  for (int d = 0; d < kPrefetch; ++d) { fetch(pf[d], fc); advance(fc); }
  int ws = 0;
  uint32_t wph = 1;           // parity to wait for on the empty barriers
  bool ok = true;
  while (cc.item < i1 && ok) {
#pragma unroll
    for (int d = 0; d < kPrefetch; ++d) {
      if (cc.item < i1 && ok) {
        ok = mbar_wait(S.wempty + 8u * ws, wph, S.abort_flag, &g_status_tc);
        if (ok) {
          const uint32_t stage = S.ring + (uint32_t)ws * P.stage_bytes;
#pragma unroll
          for (int u = 0; u < kUnits; ++u) {
            const int rr = u >> gs_log, kk = u & (gs - 1);
            const int row = row0 + 128 * rr;
            const int jj = grp * gs + kk;
            const int j = cc.st * P.mps + jj;
            const int co = cc.slab * P.NT + row;
            if (rr < nrows && row < P.NT && co < P.Co && j < P.nsteps) {
              const bool two = S.table[j].gw2 != 0xFFFFFFFFu;
              uint32_t v[4];
              const uint32_t a = stage + (uint32_t)(2 * jj) * b_lbo + (uint32_t)row * 16u;
              expand_signs<false>(pf[d][2 * u], v);
              sts128(a, v[0], v[1], v[2], v[3]);
              expand_signs<false>(pf[d][2 * u + 1], v);
              if (!two) { v[0] = 0u; v[1] = 0u; v[2] = 0u; v[3] = 0u; }
              sts128(a + b_lbo, v[0], v[1], v[2], v[3]);
            }
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(S.wfull + 8u * ws);
          if (++ws == P.stages) { ws = 0; wph ^= 1u; }
          advance(cc);
          fetch(pf[d], fc);
          advance(fc);
        }
      }
    }
  }
}

// ------------------------------------------------------------------ patch producers (2 warps)
// Granule = (phase plane, stream position, group of up to 4 channel words).
constexpr int kGranBatch = 4;

__device__ void patch_role(const TcParams &P, const Smem &S, long long i0, long long i1, int pt,
                           int lane) {
  const int tile0 = (int)(i0 / P.nslabs), tile1 = (int)((i1 - 1) / P.nslabs);
  const int s = P.stride, phases = s * s;
  const int wgroups = (P.Cw + 3) >> 2;
  const int ngran = phases * P.ppix * wgroups;
  const uint32_t plane_bytes = (uint32_t)P.ppix * 16u;
  const bool vec = (P.Cw & 3) == 0;
  int pb = 0;
  uint32_t pph = 1;
  bool ok = true;
  for (int tile = tile0; tile <= tile1 && ok; ++tile) {
    ok = mbar_wait(S.pempty + 8u * pb, pph, S.abort_flag, &g_status_tc);
    if (!ok) break;
    const uint32_t patch = S.patch + (uint32_t)pb * P.patch_bytes;
    const long long m0 = (long long)tile * kTileM;
    for (int g0 = pt; g0 < ngran; g0 += kPatThreads * kGranBatch) {
      uint32_t wv[kGranBatch][4];
      uint32_t dst[kGranBatch];
      int w0s[kGranBatch];
#pragma unroll
      for (int b = 0; b < kGranBatch; ++b) {
        const int g = g0 + b * kPatThreads;
        wv[b][0] = wv[b][1] = wv[b][2] = wv[b][3] = 0u;
        dst[b] = 0u;
        w0s[b] = -1;
        if (g < ngran) {
          // g = (phase * wgroups + wg) * ppix + q : consecutive threads take consecutive pixels
          const int pw = g / P.ppix, q = g - pw * P.ppix;
          const int phase = pw / wgroups, wg = pw - phase * wgroups;
          const int w0 = wg * 4;
          w0s[b] = w0;
          dst[b] = patch + (uint32_t)(phase * P.Cw + w0) * plane_bytes + (uint32_t)q * 16u;
          const long long sq = m0 + q;
          if (sq < P.L) {
            const long long r = sq / P.Wq;
            const int c = (int)(sq - r * P.Wq);
            const long long n = r / P.Hq;
            const int ry = (int)(r - n * P.Hq);
            const int py = phase / s, px = phase - py * s;
            const int iy = (ry - P.leadY) * s + py, ix = (c - P.leadX) * s + px;
            if (ry >= P.leadY && c >= P.leadX && iy < P.H && ix < P.W) {
              const uint32_t *src = P.xp + (((size_t)n * P.H + iy) * P.W + ix) * P.Cw + w0;
              if (vec) {
                const uint4 t = __ldg(reinterpret_cast<const uint4 *>(src));
                wv[b][0] = t.x; wv[b][1] = t.y; wv[b][2] = t.z; wv[b][3] = t.w;
              } else {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                  if (w0 + i < P.Cw) wv[b][i] = __ldg(src + i);
              }
              w0s[b] = w0 | 0x40000000;      // marks a real pixel
            }
          }
        }
      }
#pragma unroll
      for (int b = 0; b < kGranBatch; ++b) {
        if (w0s[b] >= 0) {
          const bool real = (w0s[b] & 0x40000000) != 0;
          const int w0 = w0s[b] & 0xFFFF;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (w0 + i < P.Cw) {
              uint32_t v[4] = {0u, 0u, 0u, 0u};
              if (real) {
                expand_signs<true>(wv[b][i], v);
                if (w0 + i == P.Cw - 1 && P.tail_mask != 0xFFFFFFFFu) {
                  // channels beyond C_in are the value 0
#pragma unroll
                  for (int r = 0; r < 4; ++r) v[r] &= ((P.tail_mask >> r) & 0x11111111u) * 0xFu;
                }
              }
              sts128(dst[b] + (uint32_t)i * plane_bytes, v[0], v[1], v[2], v[3]);
            }
          }
        }
      }
    }
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) mbar_arrive(S.pfull + 8u * pb);
    if (++pb == P.npb) { pb = 0; pph ^= 1u; }
  }
}

// ------------------------------------------------------------------ epilogue (8 warps)
// Warp w reads tensor-memory lanes 32 (w & 3) .. +31 (pixels) and one half of the
// slab's columns (filters).  Lane = pixel, so for one filter a warp stores 32
// consecutive stream pixels: a contiguous run of the NCHW output row.
__device__ void epilogue_role(const TcParams &P, const Smem &S, long long i0, long long i1,
                              uint32_t tmem_base, int warp, int lane) {
  const int quarter = warp & 3, half = warp >> 2;
  const int nblk = P.NT / 16;
  const int b_begin = half == 0 ? 0 : (nblk + 1) / 2;
  const int b_end = half == 0 ? (nblk + 1) / 2 : nblk;
  const size_t HoWo = (size_t)P.Ho * P.Wo;
  const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
  int tile = (int)(i0 / P.nslabs), slab = (int)(i0 - (long long)tile * P.nslabs);
  bool new_tile = true, valid = false, ok = true;
  float kv = 0.0f;
  size_t obase = 0;                       // offset of (image, filter 0, pixel)
  long long k = 0;
  for (long long item = i0; item < i1 && ok; ++item, ++k) {
    if (new_tile) {
      const long long m = (long long)tile * kTileM + quarter * 32 + lane;
      valid = m < P.L;
      if (valid) {
        const long long r = m / P.Wq;
        const int ox = (int)(m - r * P.Wq);
        const long long n = r / P.Hq;
        const int oy = (int)(r - n * P.Hq);
        valid = ox < P.Wo && oy < P.Ho;
        if (valid) {
          const size_t pix = (size_t)oy * P.Wo + ox;
          kv = __ldg(P.K + (size_t)n * HoWo + pix);
          obase = (size_t)n * P.Co * HoWo + pix;
        }
      }
    }
    const int ab = (int)(k % P.nacc);
    const uint32_t use = (uint32_t)(k / P.nacc);
    ok = mbar_wait(S.afull + 8u * ab, use & 1u, S.abort_flag, &g_status_tc);
    if (!ok) break;
    tc_fence_after();
    const uint32_t t_acc = t_lane + (uint32_t)(ab * P.NT);
    const int co0 = slab * P.NT;

    auto emit = [&](int b, const int32_t r[16]) {
      if (!valid) return;
      const int co = co0 + b * 16;
      float *op = P.out + obase + (size_t)co * HoWo;
      if (co + 16 <= P.Co && P.residual == nullptr && P.acc_out == nullptr) {
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4) {
          const float4 al = __ldg(reinterpret_cast<const float4 *>(P.alpha + co) + j4);
          const float a4[4] = {al.x, al.y, al.z, al.w};
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            *op = __fmul_rn(__fmul_rn(__int_as_float(r[j4 * 4 + jj]), kv), a4[jj]);
            op += HoWo;
          }
        }
      } else {
        const size_t o0 = obase + (size_t)co * HoWo;
        float res[16];
        if (P.residual) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            res[j] = co + j < P.Co ? P.residual[o0 + (size_t)j * HoWo] : 0.0f;
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          if (co + j < P.Co) {
            const float d = __int_as_float(r[j]);
            float v = __fmul_rn(__fmul_rn(d, kv), __ldg(P.alpha + co + j));
            if (P.residual) v += res[j];
            P.out[o0 + (size_t)j * HoWo] = v;
            if (P.acc_out) P.acc_out[o0 + (size_t)j * HoWo] = __float2int_rn(d);
          }
        }
      }
    };

    // two register sets: the load of the next 16 columns is in flight while the
    // current 16 are scaled and stored
    int32_t ra[16], rb[16];
    if (b_begin < b_end) {
      tmem_ld16(t_acc + (uint32_t)(b_begin * 16), ra);
      tmem_wait16(ra);
    }
    for (int b = b_begin; b < b_end; b += 2) {
      const bool more1 = b + 1 < b_end, more2 = b + 2 < b_end;
      if (more1) tmem_ld16(t_acc + (uint32_t)((b + 1) * 16), rb);
      else {                                     // ra was the last load: release the buffer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(S.aempty + 8u * ab);
      }
      emit(b, ra);
      if (more1) {
        tmem_wait16(rb);
        if (more2) {
          tmem_ld16(t_acc + (uint32_t)((b + 2) * 16), ra);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(S.aempty + 8u * ab);
        }
        emit(b + 1, rb);
        if (more2) tmem_wait16(ra);
      }
    }
    if (b_begin >= b_end) {                      // a warp with no columns still releases
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(S.aempty + 8u * ab);
    }
    new_tile = false;
    if (++slab == P.nslabs) { slab = 0; ++tile; new_tile = true; }
  }
}

__global__ void __launch_bounds__(kThreads, 1) binconv_tc_kernel(const TcParams P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Smem S = carve(smem, P);

  if (tid == 0) {
    for (int i = 0; i < kMaxStages; ++i) {
      mbar_init(S.wfull + 8u * i, kWgtWarps);
      mbar_init(S.wempty + 8u * i, 1);
    }
    for (int i = 0; i < kMaxPatchBufs; ++i) {
      mbar_init(S.pfull + 8u * i, kPatWarps);
      mbar_init(S.pempty + 8u * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(S.afull + 8u * i, 1);
      mbar_init(S.aempty + 8u * i, kEpiWarps);
    }
    *S.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(S.tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // the table of K-steps, once per CTA
  {
    KStep *table = reinterpret_cast<KStep *>(smem + P.off_table);
    for (int j = tid; j < P.nsteps; j += kThreads) {
      KStep ks;
      build_kstep(P, j, ks);
      table[j] = ks;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *S.tmem_slot;
  if (warp < 4) {
    // unit block scales (ue8m0 1.0 = 0x7F) in every lane of the scale columns
    const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)kSfCol;
    const uint32_t one = 0x7F7F7F7Fu;
#pragma unroll
    for (int k = 0; k < (kTmemCols - kSfCol) / 8; ++k)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};"
                   ::"r"(taddr + 8u * k), "r"(one) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  // this CTA's contiguous range of work items; item = tile * nslabs + slab
  const long long total = (long long)P.ntiles * P.nslabs;
  const long long i0 = total * blockIdx.x / gridDim.x;
  const long long i1 = total * (blockIdx.x + 1) / gridDim.x;
  if (i0 < i1) {
    if (warp < kEpiWarps) epilogue_role(P, S, i0, i1, tmem_base, warp, lane);
    else if (warp == kMmaWarp) mma_role(P, S, i0, i1, tmem_base, lane);
    else if (warp < kPatWarp0) weight_role(P, S, i0, i1, tid - 32 * kWgtWarp0, lane);
    else patch_role(P, S, i0, i1, tid - 32 * kPatWarp0, lane);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
  }
}

int floor_div(int a, int b) { return a >= 0 ? a / b : -((-a + b - 1) / b); }

struct Plan {
  TcParams P;
  size_t smem;
  bool ok;
};

Plan make_plan(const ConvGeom &g) {
  Plan pl{};
  pl.ok = false;
  TcParams &P = pl.P;
  const int s = g.stride;
  if (s < 1 || s > 2 || g.Ho < 1 || g.Wo < 1) return pl;
  P.N = g.N; P.C = g.C; P.H = g.H; P.W = g.W; P.Co = g.Co; P.kh = g.kh; P.kw = g.kw;
  P.stride = s; P.pad = g.pad; P.Ho = g.Ho; P.Wo = g.Wo; P.Cw = g.Cw;
  // stream geometry of a phase plane (see the header comment)
  P.dymin = floor_div(-g.pad, s); P.dxmin = floor_div(-g.pad, s);
  const int dymax = floor_div(g.kh - 1 - g.pad, s), dxmax = floor_div(g.kw - 1 - g.pad, s);
  P.leadY = -P.dymin; P.leadX = -P.dxmin;
  const int Hc = (g.H + s - 1) / s, Wc = (g.W + s - 1) / s;    // rows/columns of the largest plane
  const int Hd = std::max(std::max(Hc, g.Ho + dymax - P.leadY), g.Ho);
  const int Wd = std::max(std::max(Wc, g.Wo + dxmax - P.leadX), g.Wo);
  P.Hq = P.leadY + Hd; P.Wq = P.leadX + Wd;
  P.L = (long long)g.N * P.Hq * P.Wq;
  if (P.L >= (1ll << 31)) return pl;
  P.ntiles = (int)((P.L + kTileM - 1) / kTileM);
  const int halo = (dymax - P.dymin) * P.Wq + (dxmax - P.dxmin);
  P.ppix = (kTileM + halo + 1 + 7) / 8 * 8;             // +1: a lone piece reads one pixel further
  P.nplanes = s * s * g.Cw;
  P.patch_bytes = (uint32_t)P.nplanes * (uint32_t)P.ppix * 16u;
  // filter slabs: as few as fit the accumulator columns, double-buffered when possible
  P.nslabs = (g.Co + 239) / 240;
  P.NT = ((g.Co + P.nslabs - 1) / P.nslabs + 15) / 16 * 16;
  P.nacc = 2 * P.NT <= kMaxAccCols ? 2 : 1;
  // K-steps
  const int taps = g.kh * g.kw, h = g.Cw / 2;
  P.nsteps = (g.Cw % 2 == 0) ? taps * h : (taps / 2) * (2 * h + 1) + (taps % 2) * (h + 1);
  if (P.nsteps < 1 || P.nsteps > kMaxSteps) return pl;
  // weight-thread mapping: rows_mod threads cover the rows, the other thread groups take
  // other K-steps of the stage
  int ntp = 16;
  while (ntp < P.NT) ntp *= 2;                          // 16 .. 256
  P.rows_mod = std::min(ntp, 128);
  const int groups = kWgtThreads / P.rows_mod;          // 1, 2, 4, 8
  P.mps = std::max(2, std::min(8, 512 / ntp));
  P.grp_steps = P.mps / groups;                         // 2 (x2 rows), 4, 4, 2, 1
  P.stage_bytes = (uint32_t)P.mps * (uint32_t)P.NT * 32u;
  // shared memory: control, table, weight ring, patch buffers
  P.off_table = (uint32_t)kCtrlBytes;
  P.off_ring = (uint32_t)((P.off_table + (size_t)P.nsteps * sizeof(KStep) + 127) / 128 * 128);
  const size_t avail = kSmemMax - P.off_ring;
  if ((size_t)P.patch_bytes + 2 * (size_t)P.stage_bytes > avail) return pl;
  // at least 2 stages and 1 patch; then patches up to 3, stages up to 6, one more patch
  int stages = 2, npb = 1;
  auto fits = [&](int st, int pb) {
    return (size_t)st * P.stage_bytes + (size_t)pb * P.patch_bytes <= avail;
  };
  while (stages < 4 && fits(stages + 1, npb)) ++stages;
  while (npb < 3 && fits(stages, npb + 1)) ++npb;
  while (stages < kMaxStages && fits(stages + 1, npb)) ++stages;
  while (npb < kMaxPatchBufs && fits(stages, npb + 1)) ++npb;
  P.stages = stages; P.npb = npb;
  P.off_patch = P.off_ring + (uint32_t)stages * P.stage_bytes;
  pl.smem = (size_t)P.off_patch + (size_t)npb * P.patch_bytes;
  // block-scaled instruction descriptor: e2m1 x e2m1, ue8m0 scales, M = 128, N = NT
  P.idesc = (1u << 7) | (1u << 10) | ((uint32_t)(P.NT >> 3) << 17) | (1u << 23) |
            ((uint32_t)(kTileM >> 4) << 24);
  const int crem = g.C - 32 * (g.Cw - 1);
  P.tail_mask = crem == 32 ? 0xFFFFFFFFu : ((1u << crem) - 1u);
  pl.ok = true;
  return pl;
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

bool umma_tc_supported(const ConvGeom &g) { return make_plan(g).ok; }

cudaError_t launch_binconv_tc(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                              const float *K, const float *residual, const ConvGeom &g,
                              float *out, int32_t *acc_out, cudaStream_t st) {
  Plan pl = make_plan(g);
  if (!pl.ok) return cudaErrorInvalidValue;
  TcParams &P = pl.P;
  P.xp = xp; P.wp = wp; P.alpha = alpha; P.K = K; P.residual = residual;
  P.out = out; P.acc_out = acc_out;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(binconv_tc_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemMax);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  const long long total = (long long)P.ntiles * P.nslabs;
  const int sms = sm_count_cached();
  const unsigned grid = (unsigned)std::min<long long>(total, sms);
  binconv_tc_kernel<<<grid, kThreads, pl.smem, st>>>(P);
  return cudaGetLastError();
}

cudaError_t read_status_tc(int *status) {
  cudaError_t e = cudaMemcpyFromSymbol(status, g_status_tc, sizeof(int));
  if (e == cudaSuccess && *status != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_status_tc, &zero, sizeof(int));
  }
  return e;
}

}  // namespace xnor
