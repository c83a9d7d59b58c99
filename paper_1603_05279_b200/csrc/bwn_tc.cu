// Binary-Weight-Network convolution (Section 3.1, Eq. 1): I * W ~ (I (+) B) alpha with real
// inputs and B = sign(W), on the 5th-generation tensor cores.
//
// The inputs are rounded once to bfloat16 and laid out as the "pixel stream" the XNOR kernel
// uses (every input row preceded by lead zero pixels, every image by lead zero rows, one
// stream per stride phase), but materialised in memory with the padding written as zeros:
//   x_stream  bf16 [phases][L][Cp],  L = N*Hq*Wq stream positions, Cp = C rounded up to 32.
// With GEMM row m = stream position of an output pixel, tap (ky,kx) reads position
// m + shift(ky,kx) of one phase: a CTA fetches the ppix = 128 + halo positions a tile touches
// ONCE, with one TMA tile copy per phase and group of 8 channels (box = 8 channels x ppix
// positions): shared memory then holds [channel group][position][16 bytes], the no-swizzle
// K-major operand layout, and every tap's A operand is that patch at a shifted start address.
// Positions beyond the tensor read as zeros (TMA bounds fill).
//
// B operand: the packed sign words of a slab of NT filters, expanded by producer warps into
// +-1 bfloat16 rows in a ring of stages (one K-step of 16 channels = two 16-byte pieces of a
// filter row).  tcgen05.mma kind::f16 (bf16 x bf16, fp32 accumulation in tensor memory): every
// product is +-x exactly; only the fp32 accumulation rounds.
//
// Roles (576 threads, persistent, one CTA per SM, items = (pixel tile, filter slab) in tile-major
// order, a contiguous range per CTA): warps 0-7 epilogue (D * alpha (+ residual) -> NCHW; two
// warps per quarter of the lanes, taking alternate groups of 16 columns), warp 8 issues the MMAs,
// warp 9 issues the TMA copies, warps 10-17 expand weights.  Every wait is
// bounded; on expiry the CTA records XNOR_ERR_TIMEOUT, stops, and frees its tensor memory.
#include <cuda.h>

#include <algorithm>

#include "bgrad.cuh"
#include "umma_common.cuh"

namespace xnor {

__device__ int g_status_bwn = 0;

namespace {

using namespace umma;

constexpr int kEpiWarps = 8;          // two per quarter of the tensor-memory lanes
constexpr int kMmaWarp = 8;
constexpr int kTmaWarp = 9;
constexpr int kWgtWarp0 = 10, kWgtWarps = 8;
constexpr int kThreads = 32 * (kWgtWarp0 + kWgtWarps);   // 576: 18 warps, 112 registers each
constexpr int kTileM = 128;
constexpr int kTmemCols = 512;
constexpr int kMaxAcc = 4;
constexpr int kMaxStages = 8;
constexpr int kMaxPatchBufs = 3;
constexpr int kMaxTaps = 121;
constexpr size_t kCtrlBytes = 1024;
constexpr size_t kSmemMax = 232448 - 1024;

struct alignas(64) BwnParams {
  CUtensorMap tmap;            // x_stream as {8 channels, Cp/8 groups, L positions, phases}
  const uint32_t *wp;
  const float *alpha, *residual;
  float *out;
  int N, C, H, W, Co, kh, kw, stride, pad, Ho, Wo, Cw;
  int Cp, cpt;                 // channels padded to 32; K-steps per tap = Cp / 16 (even)
  int Hq, Wq, leadY, leadX;
  long long L;
  int ntiles, nslabs, NT, nacc, ppix, npb, stages, mps, nsteps, ntaps, phases;
  int tpi;                     // pixel tiles per work item (1 or 2): every weight stage then serves
                               // tpi MMAs, so the filter rows are expanded once per tpi * 128 pixels;
                               // ntiles counts items' worth of tiles (groups of tpi stream tiles)
  int nload, box_pos;          // TMA copies per operand plane of a patch and their extent in positions
  int rows_mod, grp_steps;
  uint32_t plane_bytes, phase_bytes, patch_bytes, stage_bytes;
  uint32_t off_vec, off_ring, off_patch;
  int vec_len;
  uint32_t idesc;
  int relu;
  uint32_t tap_lo[kMaxTaps];   // per tap: start of its A operand inside a patch, in 16-byte units
  uint32_t div_wq_m, div_hq_m;
  int div_wq_s, div_hq_s;
};

__device__ __forceinline__ uint32_t fast_div(uint32_t n, uint32_t m, int s) {
  return (uint32_t)(((uint64_t)n * m) >> (31 + s));
}

__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred = 0;
  asm volatile(
      "{\n\t.reg .b32 rx;\n\t.reg .pred px;\n\t"
      "elect.sync rx|px, %1;\n\t"
      "@px mov.s32 %0, 1;\n\t}"
      : "+r"(pred) : "r"(0xFFFFFFFFu));
  return pred;
}

// One MMA of 128 x NT x 16 (bf16).  One elected lane of the issuing warp runs the whole issue
// loop (a predicate per MMA in a converged warp costs a divergence each time).
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi,
                                          uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void commit_one(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar) : "memory");
}

// TMA tile copy global -> shared of one operand plane of a patch: box {8, 1, ppix, 1} at
// coordinates {0, group, pos, phase}; its bytes complete on `bar`.  The innermost coordinate
// is 0, so the copy starts on a 16-byte boundary whatever `pos` is.
__device__ __forceinline__ void tma_load_plane(uint32_t dst, const CUtensorMap *tmap, int group,
                                               int pos, int phase, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(tmap), "r"(0), "r"(group), "r"(pos), "r"(phase), "r"(bar) : "memory");
}

__device__ __forceinline__ float4 lds_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float lds_f(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}

struct Smem {
  uint32_t wfull, wempty, pfull, pempty, afull, aempty;
  uint32_t *tmem_slot;
  volatile int *abort_flag;
  uint32_t ring, patch, alpha;
};

__device__ __forceinline__ Smem carve(uint8_t *smem, const BwnParams &P) {
  Smem s;
  const uint32_t base = smem_u32(smem);
  s.wfull = base;
  s.wempty = s.wfull + 8u * kMaxStages;
  s.pfull = s.wempty + 8u * kMaxStages;
  s.pempty = s.pfull + 8u * kMaxPatchBufs;
  s.afull = s.pempty + 8u * kMaxPatchBufs;
  s.aempty = s.afull + 8u * kMaxAcc;
  s.tmem_slot = reinterpret_cast<uint32_t *>(smem + 8 * (2 * kMaxStages + 2 * kMaxPatchBufs + 2 * kMaxAcc));
  s.abort_flag = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
  s.ring = base + P.off_ring;
  s.patch = base + P.off_patch;
  s.alpha = base + P.off_vec;
  return s;
}

__device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag, &g_status_bwn));
}

// ------------------------------------------------------------------ MMA issuer (one thread)
__device__ void mma_loop(const BwnParams &P, const Smem &S, long long i0, long long i1,
                         uint32_t tmem_base) {
  const int nst = (P.nsteps + P.mps - 1) / P.mps;
  const uint32_t b_lbo = (uint32_t)P.NT * 16u;
  const uint32_t desc_hi = (128u >> 4) | (1u << 14);      // 128 B between 8-row groups; version
  const uint32_t a_lbo_hi = (P.plane_bytes >> 4) << 16;    // the K-step's second piece: next plane
  const uint32_t b_lo0 = ((S.ring & 0x3FFFFu) >> 4) | ((b_lbo >> 4) << 16);
  const uint32_t b_step = (2u * b_lbo) >> 4;
  const uint32_t a_step = (2u * P.plane_bytes) >> 4;       // next 16 channels of the same tap
  const uint32_t stage_step = P.stage_bytes >> 4;
  int ws = 0, pb = 0, ab = 0;
  uint32_t wph = 0, pph = 0, aph = 1u;
  int slab = (int)(i0 % P.nslabs);
  bool ok = true, new_tile = true;
  uint32_t patch_lo = 0;
  const uint32_t nitems = (uint32_t)(i1 - i0);
  for (uint32_t it = 0; it < nitems && ok; ++it) {
    if (new_tile) {
      ok = mbar_wait(S.pfull + 8u * pb, pph, S.abort_flag, &g_status_bwn);
      if (!ok) break;
      patch_lo = ((S.patch + (uint32_t)pb * P.patch_bytes) & 0x3FFFFu) >> 4;
    }
    ok = mbar_wait(S.aempty + 8u * ab, aph, S.abort_flag, &g_status_bwn);
    if (!ok) break;
    tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)(ab * P.tpi * P.NT);
    int tap = 0, c16 = 0;                    // K-step j = tap * cpt + c16
    for (int st = 0; st < nst && ok; ++st) {
      const int j0 = st * P.mps;
      const int nj = min(P.mps, P.nsteps - j0);
      ok = mbar_wait(S.wfull + 8u * ws, wph, S.abort_flag, &g_status_bwn);
      if (!ok) break;
      tc_fence_after();
      const uint32_t b_lo = b_lo0 + (uint32_t)ws * stage_step;
      for (int jj = 0; jj < nj; ++jj) {
        const uint32_t a_lo = ((patch_lo + P.tap_lo[tap] + (uint32_t)c16 * a_step) & 0x3FFFu) | a_lbo_hi;
        umma_bf16(d_tmem, a_lo, desc_hi, b_lo + (uint32_t)jj * b_step, desc_hi, P.idesc,
                  (j0 + jj) == 0 ? 0u : 1u);
        // the item's second pixel tile: the same patch 128 positions (128 x 16 bytes) further,
        // the same filter rows, the next accumulator
        if (P.tpi == 2)
          umma_bf16(d_tmem + (uint32_t)P.NT, a_lo + (uint32_t)kTileM, desc_hi,
                    b_lo + (uint32_t)jj * b_step, desc_hi, P.idesc, (j0 + jj) == 0 ? 0u : 1u);
        if (++c16 == P.cpt) { c16 = 0; ++tap; }
      }
      commit_one(S.wempty + 8u * ws);
      if (++ws == P.stages) { ws = 0; wph ^= 1u; }
    }
    if (!ok) break;
    new_tile = false;
    if (++slab == P.nslabs) { slab = 0; new_tile = true; }
    commit_one(S.afull + 8u * ab);
    if (new_tile || it + 1 == nitems) commit_one(S.pempty + 8u * pb);
    if (new_tile) { if (++pb == P.npb) { pb = 0; pph ^= 1u; } }
    if (++ab == P.nacc) { ab = 0; aph ^= 1u; }
  }
}

__device__ __forceinline__ void mma_role(const BwnParams &P, const Smem &S, long long i0, long long i1,
                                         uint32_t tmem_base) {
  if (elect_one()) mma_loop(P, S, i0, i1, tmem_base);
  __syncwarp();
}

// ------------------------------------------------------------------ TMA producer (one warp)
__device__ void tma_role(const BwnParams &P, const Smem &S, long long i0, long long i1, int lane) {
  const int tile0 = (int)(i0 / P.nslabs);
  const uint32_t npatches = (uint32_t)((i1 - 1) / P.nslabs) - (uint32_t)tile0 + 1u;
  bool ok = true;
  uint32_t started = 0;
  for (uint32_t seq = 0; seq < npatches && ok; ++seq) {
    const uint32_t pb = seq % (uint32_t)P.npb, use = seq / (uint32_t)P.npb;
    ok = wait_warp(S.pempty + 8u * pb, (use & 1u) ^ 1u, S.abort_flag);
    if (!ok) break;
    if (lane == 0) {
      const uint32_t bar = S.pfull + 8u * pb;
      const uint32_t dst = S.patch + pb * P.patch_bytes;
      mbar_arrive_expect_tx(bar, P.patch_bytes);
      const int pos = (tile0 + (int)seq) * P.tpi * kTileM;
      const int ngroups = P.Cp / 8;
      for (int ph = 0; ph < P.phases; ++ph)
        for (int g8 = 0; g8 < ngroups; ++g8)
          for (int ld = 0; ld < P.nload; ++ld)
            tma_load_plane(dst + (uint32_t)ph * P.phase_bytes + (uint32_t)g8 * P.plane_bytes +
                               (uint32_t)(ld * P.box_pos) * 16u,
                           &P.tmap, g8, pos + ld * P.box_pos, ph, bar);
    }
    started = seq + 1u;
  }
  if (!ok && started > 0u) {
    // gave up: the copies started last must land before the CTA's shared memory is released
    for (uint32_t back = 1; back <= (uint32_t)P.npb && back <= started; ++back) {
      const uint32_t c = started - back;
      for (int i = 0; i < (1 << 20) &&
                      !mbar_try(S.pfull + 8u * (c % (uint32_t)P.npb), (c / (uint32_t)P.npb) & 1u); ++i) {}
    }
  }
}

// ------------------------------------------------------------------ weight producers (8 warps)
// Byte kByte of a packed word (eight sign bits, a set bit is +1) -> eight bfloat16 values +-1
// (0x3F80 / 0xBF80), channel 2i in the low half of register i.  `inv` is the complemented word:
// its bit is the sign bit of the value.  Four operations per register, all shifts constant.
template <int kByte>
__device__ __forceinline__ void expand_byte(uint32_t inv, uint32_t v[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    constexpr int base = 8 * kByte;
    const int p = base + 2 * i;                         // bit of the low value; p + 1 of the high one
    const uint32_t lo = p <= 15 ? (inv << (15 - p)) : (inv >> (p - 15));
    const uint32_t hi = inv << (30 - p);
    v[i] = 0x3F803F80u | (lo & 0x8000u) | (hi & 0x80000000u);
  }
}

// A stage holds mps K-steps (mps / 2 packed words) of NT filter rows: piece (2 jj + half) of
// NT x 16 bytes.  K-step j is bits 16 (j & 1) .. + 15 of packed word j >> 1 of the filter (the
// channels are padded to whole words), so a word expands to four consecutive pieces.  Thread
// mapping: row = wt % rows_mod, the 256 / rows_mod groups split the words of a stage (at most
// two words per thread and stage).  The words of the NEXT stage are fetched before the current
// one is expanded: the filters are re-read (from L2) for every work item.
__device__ void weight_role(const BwnParams &P, const Smem &S, long long i0, long long i1, int wt,
                            int lane) {
  constexpr int kMaxWords = 2;
  const int nst = (P.nsteps + P.mps - 1) / P.mps;
  const int wps = P.mps >> 1, nwords = P.nsteps >> 1;   // words per stage, per filter row
  const int row = wt % P.rows_mod, grp = wt / P.rows_mod;
  const int wpt = P.grp_steps;                          // words per thread and stage (1 or 2)
  const bool grp_on = grp * wpt < wps && row < P.NT;
  const uint32_t b_lbo = (uint32_t)P.NT * 16u;
  auto fetch = [&](int st, int co, uint32_t w[kMaxWords]) {
#pragma unroll
    for (int u = 0; u < kMaxWords; ++u) {
      const int wl = grp * wpt + u, f = st * wps + wl;
      w[u] = 0u;
      if (grp_on && u < wpt && wl < wps && f < nwords && co < P.Co)
        w[u] = __ldg(P.wp + packed_weight_index(P.Co, co, f));
    }
  };
  int ws = 0;
  uint32_t wph = 1u;
  bool ok = true;
  int slab = (int)(i0 % P.nslabs);
  uint32_t cur[kMaxWords], nxt[kMaxWords];
  fetch(0, slab * P.NT + row, cur);
  for (long long it = i0; it < i1 && ok; ++it) {
    int nslab = slab + 1;
    if (nslab == P.nslabs) nslab = 0;
    for (int st = 0; st < nst && ok; ++st) {
      // the stage after this one: the next of this item, or the first of the next item
#pragma unroll
      for (int u = 0; u < kMaxWords; ++u) nxt[u] = 0u;
      if (st + 1 < nst) fetch(st + 1, slab * P.NT + row, nxt);
      else if (it + 1 < i1) fetch(0, nslab * P.NT + row, nxt);
      ok = mbar_wait_relaxed(S.wempty + 8u * ws, wph, S.abort_flag, &g_status_bwn, 50);
      if (!ok) break;
      if (grp_on) {
        const uint32_t stage = S.ring + (uint32_t)ws * P.stage_bytes + (uint32_t)row * 16u;
#pragma unroll
        for (int u = 0; u < kMaxWords; ++u) {
          const int wl = grp * wpt + u;
          if (u < wpt && wl < wps && st * wps + wl < nwords) {
            const uint32_t inv = ~cur[u];
            const uint32_t a = stage + (uint32_t)(4 * wl) * b_lbo;       // pieces 4 wl .. 4 wl + 3
            uint32_t v[4];
            expand_byte<0>(inv, v); sts128(a, v[0], v[1], v[2], v[3]);
            expand_byte<1>(inv, v); sts128(a + b_lbo, v[0], v[1], v[2], v[3]);
            expand_byte<2>(inv, v); sts128(a + 2u * b_lbo, v[0], v[1], v[2], v[3]);
            expand_byte<3>(inv, v); sts128(a + 3u * b_lbo, v[0], v[1], v[2], v[3]);
          }
        }
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(S.wfull + 8u * ws);
      if (++ws == P.stages) { ws = 0; wph ^= 1u; }
#pragma unroll
      for (int u = 0; u < kMaxWords; ++u) cur[u] = nxt[u];
    }
    slab = nslab;
  }
}

// ------------------------------------------------------------------ epilogue (8 warps)
// A warp reads tensor-memory lanes 32 q .. + 31 (stream positions) of its quarter q and the
// groups of 16 columns (filters) e, e + 2, ...; for one filter a warp stores 32 consecutive
// pixels of the NCHW output.
__device__ void epilogue_role(const BwnParams &P, const Smem &S, long long i0, long long i1,
                              uint32_t tmem_base, int quarter, int e, int lane) {
  const int b_end = P.NT / 16;
  const int nk = (b_end - e + 1) / 2;                 // groups of this warp per item
  const size_t HoWo = (size_t)P.Ho * P.Wo;
  const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
  const bool relu = P.relu != 0;
  int tile = (int)(i0 / P.nslabs), slab = (int)(i0 - (long long)tile * P.nslabs);
  struct Pix { bool valid; size_t obase; };
  auto decode = [&](int t) {
    Pix px{false, 0};
    const uint32_t m = (uint32_t)t * kTileM + (uint32_t)(quarter * 32 + lane);
    if (m < (uint32_t)P.L) {
      const uint32_t r = fast_div(m, P.div_wq_m, P.div_wq_s);
      const int ox = (int)(m - r * (uint32_t)P.Wq);
      const uint32_t n = fast_div(r, P.div_hq_m, P.div_hq_s);
      const int oy = (int)(r - n * (uint32_t)P.Hq);
      if (ox < P.Wo && oy < P.Ho) {
        px.valid = true;
        px.obase = (size_t)n * P.Co * HoWo + (size_t)oy * P.Wo + ox;
      }
    }
    return px;
  };
  int ab = 0;
  uint32_t fph = 0;
  bool ok = true;
  const uint32_t nitems = (uint32_t)(i1 - i0);
  for (uint32_t it = 0; it < nitems && ok; ++it) {
    ok = mbar_wait_relaxed(S.afull + 8u * ab, fph, S.abort_flag, &g_status_bwn, 200);
    if (!ok) break;
    tc_fence_after();
    const int co0 = slab * P.NT;
    if (nk == 0) {                               // a slab of 16 filters: nothing for the second warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(S.aempty + 8u * ab);
    }
   for (int tt = 0; tt < P.tpi && nk > 0; ++tt) {   // the item's pixel tiles, one accumulator each
    const Pix px = decode(tile * P.tpi + tt);
    const bool last_tile = tt + 1 == P.tpi;
    const uint32_t t_acc = t_lane + (uint32_t)((ab * P.tpi + tt) * P.NT);
    int32_t nx[16], cur[16];
    tmem_ld16(t_acc + (uint32_t)(e * 16), nx);
#pragma unroll 1
    for (int k = 0; k < nk; ++k) {
      const int b = e + 2 * k;
      tmem_wait16(nx);
#pragma unroll
      for (int j = 0; j < 16; ++j) cur[j] = nx[j];
      if (k + 1 < nk) {
        tmem_ld16(t_acc + (uint32_t)((b + 2) * 16), nx);
      } else if (last_tile) {                    // last load of the item done: release its accumulators
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(S.aempty + 8u * ab);
      }
      if (!px.valid) continue;
      const int co = co0 + b * 16;
      const size_t o0 = px.obase + (size_t)co * HoWo;
      if (co + 16 <= P.Co && P.residual == nullptr && HoWo < ((size_t)1 << 27)) {
        // whole group, no residual: 32-bit offsets from one pointer
        float *op = P.out + o0;
        const uint32_t howo = (uint32_t)HoWo;
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4) {
          const float4 al = lds_f4(S.alpha + (uint32_t)(co * 4 + j4 * 16));
          const float a4[4] = {al.x, al.y, al.z, al.w};
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const float v = __fmul_rn(__int_as_float(cur[j4 * 4 + jj]), a4[jj]);
            op[(uint32_t)(j4 * 4 + jj) * howo] = relu ? fmaxf(v, 0.0f) : v;
          }
        }
        continue;
      }
      float res[16];
      if (P.residual != nullptr) {
#pragma unroll
        for (int j = 0; j < 16; ++j) res[j] = co + j < P.Co ? P.residual[o0 + (size_t)j * HoWo] : 0.0f;
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (co + j < P.Co) {
          float v = __fmul_rn(__int_as_float(cur[j]), lds_f(S.alpha + (uint32_t)((co + j) * 4)));
          if (P.residual != nullptr) v += res[j];
          if (relu) v = fmaxf(v, 0.0f);
          P.out[o0 + (size_t)j * HoWo] = v;
        }
      }
    }
   }
    if (++slab == P.nslabs) { slab = 0; ++tile; }
    if (++ab == P.nacc) { ab = 0; fph ^= 1u; }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
bwn_conv_kernel(const __grid_constant__ BwnParams P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Smem S = carve(smem, P);
  if (tid == 0) {
    for (int i = 0; i < kMaxStages; ++i) {
      mbar_init(S.wfull + 8u * i, kWgtWarps);
      mbar_init(S.wempty + 8u * i, 1);
    }
    for (int i = 0; i < kMaxPatchBufs; ++i) {
      mbar_init(S.pfull + 8u * i, 1);
      mbar_init(S.pempty + 8u * i, 1);
    }
    for (int i = 0; i < kMaxAcc; ++i) {
      mbar_init(S.afull + 8u * i, 1);
      mbar_init(S.aempty + 8u * i, kEpiWarps);
    }
    *S.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < P.vec_len; i += kThreads)
    reinterpret_cast<float *>(smem + P.off_vec)[i] =
        i < P.Co ? (P.alpha != nullptr ? __ldg(P.alpha + i) : 1.0f) : 0.0f;   // no alpha: unit scale
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(S.tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *S.tmem_slot;

  const long long total = (long long)P.ntiles * P.nslabs;
  const long long i0 = total * blockIdx.x / gridDim.x;
  const long long i1 = total * (blockIdx.x + 1) / gridDim.x;
  if (i0 < i1) {
    if (warp < kEpiWarps) epilogue_role(P, S, i0, i1, tmem_base, warp & 3, warp >> 2, lane);
    else if (warp == kMmaWarp) mma_role(P, S, i0, i1, tmem_base);
    else if (warp == kTmaWarp) tma_role(P, S, i0, i1, lane);
    else weight_role(P, S, i0, i1, tid - 32 * kWgtWarp0, lane);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
}

// ------------------------------------------------------------------ input preparation
// fp32 NCHW (after the optional BatchNorm affine) -> bf16 stream [phase][position][Cp], zeros at
// padding positions and in channels C .. Cp - 1.  A block handles 32 consecutive stream
// positions of one phase, 64 channels at a time: reads run along the positions (consecutive
// input pixels, eight loads per thread in flight), writes along the channels (a lane packs two
// channels, a warp writes the 128 bytes of a position); the transposition goes through shared
// memory.
__device__ __forceinline__ uint32_t bf16_rne(float v) {
  // round to nearest even on the bit pattern (NaN and infinity pass through truncated)
  uint32_t u = __float_as_uint(v);
  if ((u & 0x7F800000u) != 0x7F800000u) u += 0x7FFFu + ((u >> 16) & 1u);
  return u >> 16;
}

__global__ void __launch_bounds__(256)
bwn_prepare_kernel(const float *__restrict__ x, const float *__restrict__ scale,
                   const float *__restrict__ shift, const float *__restrict__ gmax, int N, int C, int H,
                   int W, int s, int Hq, int Wq, int leadY, int leadX, long long L, int Cp,
                   uint16_t *__restrict__ xs) {
  __shared__ float tile[64][33];
  const int lane = threadIdx.x & 31, wy = threadIdx.x >> 5;      // 8 warps
  const long long nblk = (L + 31) / 32;
  const int phase = (int)(blockIdx.x / nblk);
  const long long m0 = (long long)(blockIdx.x - phase * nblk) * 32;
  const int py = phase / s, px = phase - py * s;
  // this lane's stream position for the reads
  const long long m = m0 + lane;
  bool real = m < L;
  size_t src = 0;
  float gm = 0.0f;             // gradient mode: the scale of this position's image
  if (real) {
    const long long r = m / Wq;
    const int c = (int)(m - r * Wq);
    const long long n = r / Hq;
    if (gmax != nullptr) gm = __ldg(gmax + n);
    const int ry = (int)(r - n * Hq);
    const int iy = (ry - leadY) * s + py, ix = (c - leadX) * s + px;
    real = ry >= leadY && c >= leadX && iy < H && ix < W;
    src = ((size_t)n * C * H + iy) * W + ix;
  }
  const size_t plane = (size_t)H * W;
  uint32_t *dst = reinterpret_cast<uint32_t *>(xs + ((size_t)phase * L + m0) * Cp);   // Cp is even
  for (int c0 = 0; c0 < Cp; c0 += 64) {
    // warp wy reads channels c0 + wy, + 8, ..., + 56 of the 32 positions
    float v[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int ch = c0 + wy + 8 * q;
      v[q] = (real && ch < C) ? __ldg(x + src + (size_t)ch * plane) : 0.0f;
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int ch = c0 + wy + 8 * q;
      if (gmax != nullptr) {
        // binarised gradient (Section 3.2, "Binary Gradient"): sign(g) scaled by the image's
        // max|g| and, here, by the filter's alpha (`scale`), the product formed in fp32
        if (real && ch < C) v[q] = v[q] >= 0.0f ? __fmul_rn(gm, __ldg(scale + ch)) : -__fmul_rn(gm, __ldg(scale + ch));
      } else if (scale != nullptr && real && ch < C) {
        v[q] = __fmaf_rn(__ldg(scale + ch), v[q], __ldg(shift + ch));
      }
      tile[wy + 8 * q][lane] = v[q];
    }
    __syncthreads();
    // warp wy writes positions wy, wy + 8, ...: lane = channels c0 + 2 lane, + 1
    if (c0 + 2 * lane < Cp) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int pos = wy + 8 * q;
        if (m0 + pos < L)
          dst[((size_t)pos * Cp + c0) / 2 + lane] =
              bf16_rne(tile[2 * lane][pos]) | (bf16_rne(tile[2 * lane + 1][pos]) << 16);
      }
    }
    __syncthreads();
  }
}

int floor_div(int a, int b) { return a >= 0 ? a / b : -((-a + b - 1) / b); }

struct BwnPlan {
  BwnParams P;
  size_t smem;
  bool ok;
};

// Stream geometry shared by the preparation kernel and the convolution.
struct StreamGeom {
  int s, phases, dymin, dxmin, dymax, dxmax, leadY, leadX, Hq, Wq, Cp;
  long long L;
};

StreamGeom stream_geom(const ConvGeom &g) {
  StreamGeom q;
  q.s = g.stride;
  q.phases = q.s * q.s;
  q.dymin = floor_div(-g.pad, q.s); q.dxmin = floor_div(-g.pad, q.s);
  q.dymax = floor_div(g.kh - 1 - g.pad, q.s); q.dxmax = floor_div(g.kw - 1 - g.pad, q.s);
  q.leadY = -q.dymin; q.leadX = -q.dxmin;
  const int Hc = (g.H + q.s - 1) / q.s, Wc = (g.W + q.s - 1) / q.s;
  const int Hd = std::max(std::max(Hc, g.Ho + q.dymax - q.leadY), g.Ho);
  const int Wd = std::max(std::max(Wc, g.Wo + q.dxmax - q.leadX), g.Wo);
  q.Hq = q.leadY + Hd; q.Wq = q.leadX + Wd;
  q.L = (long long)g.N * q.Hq * q.Wq;
  q.Cp = (g.C + 31) / 32 * 32;      // whole packed words: K-step j is half j & 1 of word j >> 1
  return q;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (no link-time dependency on
// the driver library).
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

BwnPlan make_plan(const ConvGeom &g) {
  BwnPlan pl{};
  pl.ok = false;
  BwnParams &P = pl.P;
  if (g.stride < 1 || g.stride > 2 || g.Ho < 1 || g.Wo < 1 || g.kh * g.kw > kMaxTaps) return pl;
  const StreamGeom q = stream_geom(g);
  P.N = g.N; P.C = g.C; P.H = g.H; P.W = g.W; P.Co = g.Co; P.kh = g.kh; P.kw = g.kw;
  P.stride = g.stride; P.pad = g.pad; P.Ho = g.Ho; P.Wo = g.Wo; P.Cw = g.Cw;
  P.Cp = q.Cp; P.cpt = q.Cp / 16;
  P.Hq = q.Hq; P.Wq = q.Wq; P.leadY = q.leadY; P.leadX = q.leadX; P.L = q.L;
  P.phases = q.phases;
  P.ntaps = g.kh * g.kw;
  P.nsteps = P.ntaps * P.cpt;
  const int halo = (q.dymax - q.dymin) * q.Wq + (q.dxmax - q.dxmin);
  if ((kTileM + halo + 7) / 8 * 8 > 256) return pl;        // a tile's window: at most one TMA box
  if (q.L + 4 * kTileM + 256 >= (1ll << 31)) return pl;
  // filter slabs: as few as fit two accumulators into the tensor-memory columns
  const int max_nt = 128;
  P.nslabs = (g.Co + max_nt - 1) / max_nt;
  P.NT = ((g.Co + P.nslabs - 1) / P.nslabs + 15) / 16 * 16;
  // weight stages: rows_mod threads cover the rows, the other groups split a stage's K-steps
  int ntp = 16;
  while (ntp < P.NT) ntp *= 2;
  P.rows_mod = ntp;
  const int groups = std::max(1, 32 * kWgtWarps / ntp);    // >= 2: slabs hold at most 128 filters
  P.mps = 8;                                               // K-steps per stage = 4 packed words per row
  P.grp_steps = std::max(1, (P.mps / 2) / groups);         // words per thread and stage: 2 or 1
  P.stage_bytes = (uint32_t)P.mps * (uint32_t)P.NT * 32u;
  P.off_vec = (uint32_t)((kCtrlBytes + 127) / 128 * 128);
  P.vec_len = (g.Co + 15) / 16 * 16 + 256;
  P.off_ring = (uint32_t)((P.off_vec + (size_t)P.vec_len * 4 + 127) / 128 * 128);
  // Two pixel tiles per work item when their common window (256 + halo positions) fits beside two
  // weight stages: the expansion of the filter rows, which bounds the kernel, is then shared by
  // two MMAs.  The window is fetched with one or two TMA copies per operand plane (box <= 256).
  const int stream_tiles = (int)((q.L + kTileM - 1) / kTileM);
  for (P.tpi = (kTmemCols / P.NT >= 2 && stream_tiles >= 2) ? 2 : 1; P.tpi >= 1; --P.tpi) {
    P.ppix = (P.tpi * kTileM + halo + 7) / 8 * 8;
    P.nload = P.ppix > 256 ? 2 : 1;
    if (P.nload == 2) P.ppix = (P.ppix + 15) / 16 * 16;   // two boxes of a multiple of 8 positions
    P.box_pos = P.ppix / P.nload;
    P.plane_bytes = (uint32_t)P.ppix * 16u;
    P.phase_bytes = P.plane_bytes * (uint32_t)(P.Cp / 8);
    P.patch_bytes = P.phase_bytes * (uint32_t)P.phases;
    if (P.off_ring + 2 * (size_t)P.stage_bytes + P.patch_bytes <= kSmemMax) break;
  }
  if (P.tpi < 1) return pl;
  P.ntiles = (stream_tiles + P.tpi - 1) / P.tpi;
  P.nacc = std::max(1, std::min(kMaxAcc, kTmemCols / (P.NT * P.tpi)));
  const size_t avail = kSmemMax - P.off_ring;
  int stages = 2, npb = 1;
  auto fits = [&](int st, int pb) { return (size_t)st * P.stage_bytes + (size_t)pb * P.patch_bytes <= avail; };
  while (stages < 4 && fits(stages + 1, npb)) ++stages;
  while (npb < 2 && fits(stages, npb + 1)) ++npb;
  while (stages < kMaxStages && fits(stages + 1, npb)) ++stages;
  while (npb < kMaxPatchBufs && fits(stages, npb + 1)) ++npb;
  P.stages = stages; P.npb = npb;
  P.off_patch = (uint32_t)((P.off_ring + (size_t)stages * P.stage_bytes + 127) / 128 * 128);
  pl.smem = (size_t)P.off_patch + (size_t)npb * P.patch_bytes;
  if (pl.smem > kSmemMax) return pl;
  // instruction descriptor: D fp32, A and B bf16, both K-major, N = NT, M = 128
  P.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.NT >> 3) << 17) |
            ((uint32_t)(kTileM >> 4) << 24);
  for (int tap = 0; tap < P.ntaps; ++tap) {
    const int ky = tap / g.kw, kx = tap - ky * g.kw;
    const int ay = ky - g.pad, ax = kx - g.pad;
    const int dy = floor_div(ay, q.s), dx = floor_div(ax, q.s);
    const int py = ay - dy * q.s, px = ax - dx * q.s;
    const int phase = py * q.s + px;
    const int shift = (dy - q.dymin) * q.Wq + (dx - q.dxmin);
    P.tap_lo[tap] = ((uint32_t)phase * P.phase_bytes + (uint32_t)shift * 16u) >> 4;
  }
  auto magic = [](uint32_t d, uint32_t *m, int *sh) {
    int l = 0;
    while ((1u << l) < d) ++l;
    *sh = l;
    *m = (uint32_t)((((unsigned long long)1 << (31 + l)) + d - 1) / d);
  };
  magic((uint32_t)P.Wq, &P.div_wq_m, &P.div_wq_s);
  magic((uint32_t)P.Hq, &P.div_hq_m, &P.div_hq_s);
  pl.ok = true;
  return pl;
}

}  // namespace

bool bwn_supported(const ConvGeom &g) { return make_plan(g).ok; }

size_t bwn_stream_elems(const ConvGeom &g) {
  if (g.stride < 1 || g.Ho < 1 || g.Wo < 1) return 0;
  const StreamGeom q = stream_geom(g);
  return (size_t)q.phases * (size_t)q.L * (size_t)q.Cp;
}

cudaError_t launch_bwn_prepare(const float *x, const float *scale, const float *shift,
                               const ConvGeom &g, uint16_t *x_stream, cudaStream_t st) {
  const StreamGeom q = stream_geom(g);
  const long long nblk = (q.L + 31) / 32 * q.phases;
  if (nblk >= (1ll << 31)) return cudaErrorInvalidValue;
  bwn_prepare_kernel<<<(unsigned)nblk, 256, 0, st>>>(x, scale, shift, nullptr, g.N, g.C, g.H, g.W, q.s,
                                                    q.Hq, q.Wq, q.leadY, q.leadX, q.L, q.Cp, x_stream);
  return cudaGetLastError();
}

cudaError_t launch_bwn_prepare_grad(const float *g, const float *alpha, const float *gmax,
                                    const ConvGeom &gb, uint16_t *g_stream, cudaStream_t st) {
  const StreamGeom q = stream_geom(gb);
  const long long nblk = (q.L + 31) / 32 * q.phases;
  if (nblk >= (1ll << 31)) return cudaErrorInvalidValue;
  bwn_prepare_kernel<<<(unsigned)nblk, 256, 0, st>>>(g, alpha, nullptr, gmax, gb.N, gb.C, gb.H, gb.W, q.s,
                                                    q.Hq, q.Wq, q.leadY, q.leadX, q.L, q.Cp, g_stream);
  return cudaGetLastError();
}

cudaError_t launch_bwn_conv(const uint16_t *x_stream, const uint32_t *wp, const float *alpha,
                            const float *residual, const ConvGeom &g, float *out, cudaStream_t st) {
  BwnPlan pl = make_plan(g);
  if (!pl.ok) return cudaErrorInvalidValue;
  BwnParams &P = pl.P;
  EncodeTiledFn encode = encode_tiled_fn();
  if (encode == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[4] = {8, (cuuint64_t)(P.Cp / 8), (cuuint64_t)P.L, (cuuint64_t)P.phases};
  const cuuint64_t strides[3] = {16, (cuuint64_t)P.Cp * 2, (cuuint64_t)P.L * P.Cp * 2};
  const cuuint32_t box[4] = {8, 1, (cuuint32_t)P.box_pos, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  if (encode(&P.tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<uint16_t *>(x_stream), dims,
             strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  P.wp = wp; P.alpha = alpha; P.residual = residual; P.out = out;
  P.relu = (g.flags & XNOR_FLAG_RELU) ? 1 : 0;
  static bool attr_flags[64] = {};
  bool &attr_set = attr_done_for_current_device(attr_flags);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(bwn_conv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemMax);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  const long long total = (long long)P.ntiles * P.nslabs;
  const unsigned grid = (unsigned)std::min<long long>(total, sm_count_of_current_device());
  bwn_conv_kernel<<<grid, kThreads, pl.smem, st>>>(P);
  cudaError_t e = cudaGetLastError();
  return e;
}

cudaError_t read_status_bwn(int *status) {
  cudaError_t e = cudaMemcpyFromSymbol(status, g_status_bwn, sizeof(int));
  if (e == cudaSuccess && *status != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_status_bwn, &zero, sizeof(int));
  }
  return e;
}

}  // namespace xnor
