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
//        warps into a ring of shared-memory stages.  One MMA (a K-step, K = 64)
//        consumes two 32-channel pieces; a piece is one packed word (tap,
//        channel word) of a filter row, and K-step j takes words 2j and 2j+1
//        of the row in memory order, so a step may straddle two taps and no
//        step is wasted on channel padding.  The host precomputes, per step,
//        the A-operand descriptor (start of the lower-addressed piece, distance
//        to the other one) and whether the two pieces are swapped.
//
//  Encodings.  A packed word holds 32 sign bits; it becomes 32 e2m1 nibbles in
//  four registers, register r holding channels r, r+4, ..., r+28.  Activations
//  are +-{2, 1, 0.5, 0.5} for r = 0..3, weights +-{0.5, 1, 2, 2}: every product
//  is the product of the two signs.
//
//  Roles (512 threads, one CTA per SM, CTAs loop over work items = (pixel
//  tile, filter slab)): warps 0-3 epilogue (tensor memory -> registers ->
//  coalesced NCHW stores of D * K * alpha (+ residual)), warp 4 issues the
//  MMAs, warps 5-12 expand weights, warps 13-15 expand activation patches.
//  Accumulators are multi-buffered in tensor memory so the epilogue of one
//  item overlaps the MMAs of the next.  Every wait is bounded: on expiry the
//  CTA records XNOR_ERR_TIMEOUT in a device status word, stops, frees its
//  tensor memory and exits.
//
//  CTA pairs (kPair kernels, clusters of 2).  One tcgen05.mma.cta_group::2
//  drives the tensor cores of two SMs: M = 256 (each CTA's 128-position tile,
//  patch and tensor memory) and each CTA expands and holds half of a slab's
//  filter rows.  The producers of both CTAs arrive on the barriers of rank 0,
//  whose MMA warp issues; its commits reach the consumer barriers of both.
//
//  Fused BinActiv (kFuse kernels).  The epilogue also applies the next layer's
//  BatchNorm affine to its output values, packs their sign bits along the
//  filters (the next layer's channels) and writes partial sums of |y|.
//
//  Two schedules.  "Resident": when the expanded rows of a filter slab fit in
//  shared memory beside two patches, the slab is expanded ONCE per CTA and the
//  CTA then walks the pixel tiles of that slab (items in slab-major order, one
//  patch per item); the weight warps, idle after the fill, join the epilogue
//  (three warps per quarter of the lanes, splitting the columns).  "Streaming":
//  otherwise the weights of every item pass through a ring of stages (items in
//  tile-major order, so that a patch serves all slabs of its tile).
#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "umma_common.cuh"

namespace xnor {

__device__ int g_status_tc = 0;

// Checking build (-DXNOR_BOUNDS_CHECK): every shared-memory address a producer computes and
// every global index the epilogue stores to is compared with the extent of its buffer; the
// first violation is recorded (its site number) and the access is skipped, so nothing traps.
// In the ordinary build in_bounds() is the constant true and its argument is never evaluated.
#ifdef XNOR_BOUNDS_CHECK
__device__ int g_bounds_tc = 0;
#define in_bounds(cond, site) ((cond) ? true : (atomicCAS(&xnor::g_bounds_tc, 0, (site)), false))
#else
#define in_bounds(cond, site) true
#endif

namespace {

using namespace umma;

// nanoseconds a waiting role sleeps between polls of its barrier
#ifndef XNOR_SLEEP_EPI
#define XNOR_SLEEP_EPI 200
#endif
#ifndef XNOR_SLEEP_PAT
#define XNOR_SLEEP_PAT 200
#endif
#ifndef XNOR_SLEEP_WGT
#define XNOR_SLEEP_WGT 50
#endif

constexpr int kEpiWarps = 4;
constexpr int kMmaWarp = 4;
constexpr int kWgtWarp0 = 5, kWgtWarps = 8;
constexpr int kPatWarp0 = 13, kPatWarps = 3;
constexpr int kThreads = 32 * (kPatWarp0 + kPatWarps);     // 512: 16 warps, 128 registers each
constexpr int kTileM = 128;          // stream positions per tile = tensor-memory lanes
constexpr int kTmemCols = 512;
constexpr int kSfCol = 480;          // columns [480, 512): unit block scales
constexpr int kMaxAccCols = 480;
constexpr int kMaxAcc = 4;           // accumulator buffers
constexpr int kMaxStages = 6;         // ring stages of the streaming schedule
constexpr int kMaxBarStages = 32;    // stage barriers (the resident schedule has one stage per mps K-steps of a row)
constexpr int kEpiSplitMax = 3;      // warps per lane quarter in the resident epilogue
constexpr int kMaxPatchBufs = 4;
constexpr int kMaxRaw = 6;            // raw buffers: up to 2 for each of up to 3 subgroups of patch warps
constexpr int kPatUnits = 2;         // patch units a warp works on together
constexpr int kMaxSteps = 800;       // K-steps (MMAs) per work item (< 1024: swap_mask)
constexpr size_t kCtrlBytes = 1024;
constexpr size_t kSmemMax = 232448 - 1024;

struct TcParams {
  const uint32_t *xp, *wp;
  const float *alpha, *K, *residual;
  float *out;
  int32_t *acc_out;
  int relu;                    // max(v, 0) on every stored value
  float out_scale;             // extra factor of D K alpha (1 unless several calls build one output), folded into the staged alpha
  int acc_shift, acc_accum;    // acc_out receives D << acc_shift, stored or added to its content
  int N, C, H, W, Co, kh, kw, stride, pad, Ho, Wo, Cw;
  int Hq, Wq, leadY, leadX;    // stream geometry of every phase plane
  int dymin, dxmin;
  long long L;                 // stream length N*Hq*Wq
  int ntiles, nslabs, NT;      // pixel tiles, filter slabs, filters per slab (multiple of 16)
  int nacc;                    // accumulator buffers in tensor memory (1 .. 4)
  int ppix;                    // stream positions staged per phase plane (128 + halo, rounded to 8)
  int nplanes;                 // stride*stride*Cw operand planes per patch
  int npb;                     // patch buffers
  int nsteps;                  // K-steps per item
  int mps;                     // K-steps per weight stage
  int stages;
  uint32_t patch_bytes, stage_bytes;
  int rows_mod, grp_steps;     // weight-thread mapping (see weight producer)
  uint32_t off_ring, off_patch, off_raw;  // byte offsets in dynamic shared memory
  uint32_t off_vec;            // per-filter vectors staged for the epilogue: alpha, then (fused)
  int vec_len;                 // the next layer's scale and shift; vec_len floats each
  uint32_t raw_bytes;          // size of a raw buffer: the packed input rows a patch can touch
  int nraw;                    // raw buffers per subgroup of patch warps (1 or 2)
  int pat_group;               // warps that build patches
  int pat_sub;                 // subgroups they form (each builds whole patches): 3 or 1
  int wgt_warps;               // warps that expand weights: 8, or 4
  uint32_t idesc;
  uint32_t tail_mask;          // bits of real channels in the last word
  // Low word of the A-operand descriptor of every K-step (start address relative to the
  // patch in bits 0-13, leading-dimension offset in bits 16-29; the high word is the same
  // for all).  It lives in the kernel parameters so that the MMA issuer reads and offsets
  // it on the uniform datapath: an MMA is as short as 32 cycles, and descriptors that pass
  // through per-thread registers cost more than that to issue.
  uint32_t adesc_lo[kMaxSteps];
  uint32_t swap_mask[32];              // bit j: word 2j+1 is the first piece of step j
  int row_words;               // packed words per filter row = k_h*k_w*Cw
  int pair;                    // 1: two CTAs (a cluster) share every MMA: 256 pixels x NT filters
  int NTh;                     // filter rows of a slab that one CTA expands and holds: NT or NT/2
  // Fused BinActiv of the next layer (kFuse kernels): the epilogue also applies the next
  // BatchNorm affine to its output values, packs their signs along the filters (the next
  // layer's channels) and sums |y| over the filters it handles.
  const float *nscale, *nshift;      // [C_out], both null = identity
  uint32_t *xp_next;                 // u32 [N][Ho][Wo][Cw_next]
  float *A_part;                     // fp32 [nslabs * epi_split][N][Ho][Wo]: partial sums of |y|
  int Cw_next;                       // ceil(C_out / 32)
  int resident;                // 1: resident schedule (stages = all stages of a slab)
  int epi_split;               // warps per lane quarter that drain an accumulator
  int any_swap;                // some bit of swap_mask is set
  uint32_t div_wq_m, div_hq_m; // multipliers and shifts of the exact divisions by Wq and Hq
  int div_wq_s, div_hq_s;      // (dividends below 2^31)
  uint32_t div_pg_m, div_g_m;  // the same for the patch units: by phases * ngrp and by ngrp
  int div_pg_s, div_g_s;       // (ngrp = groups of four channel words)
};

// One MMA.  The issuing warp elects one lane, and that lane alone runs the whole issue loop:
// a predicate per MMA inside a converged warp costs a divergence and a reconvergence each
// time (measured: 95 cycles per MMA against 65 for the single-thread loop, the tensor core
// needing 64 for 128 x 128 x 64).  Descriptors are passed as their two 32-bit halves.
__device__ __forceinline__ void umma_mxf4(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi,
                                          uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                          uint32_t sf, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], da, db, %5, [%7], [%7], p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate),
        "r"(sf)
      : "memory");
}

__device__ __forceinline__ void umma_commit_one(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar) : "memory");
}

// The same for a CTA pair: one instruction drives the tensor cores of both SMs (M = 256: rows
// 0-127 from this CTA's patch into its tensor memory, rows 128-255 the peer's; each CTA
// supplies half of the N filter rows).  Commits signal the barrier at the same offset in both.
__device__ __forceinline__ void umma_mxf4_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi,
                                               uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                               uint32_t sf, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.block32 [%0], da, db, %5, [%7], [%7], p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate),
        "r"(sf)
      : "memory");
}

__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .b16 mask;\n\t"
      "mov.b16 mask, 3;\n\t"
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], mask;\n\t}"
      ::"r"(bar) : "memory");
}

template <bool kPair>
__device__ __forceinline__ void umma_issue(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi,
                                           uint32_t b_lo, uint32_t b_hi, uint32_t idesc, uint32_t sf,
                                           uint32_t accumulate) {
  if (kPair) umma_mxf4_pair(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, sf, accumulate);
  else umma_mxf4(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, sf, accumulate);
}

template <bool kPair>
__device__ __forceinline__ void umma_commit_to(uint32_t bar) {
  if (kPair) umma_commit_pair(bar);
  else umma_commit_one(bar);
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

// Shift of a filter tap inside a phase plane, and the plane it reads.
inline void tap_geometry(const TcParams &P, int tap, int &phase, int &shift) {
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
inline uint32_t piece_offset(const TcParams &P, int tap, int w) {
  int phase, shift;
  tap_geometry(P, tap, phase, shift);
  return (uint32_t)(phase * P.Cw + w) * ((uint32_t)P.ppix * 16u) + (uint32_t)shift * 16u;
}

// K-step j: pieces = words 2j and 2j+1 of a filter row (flat index tap*Cw + w).  Returns
// the low descriptor word of its A operand; *swap tells whether word 2j+1 comes first.
inline uint32_t kstep_desc(const TcParams &P, int j, bool *swap) {
  const int f1 = 2 * j, f2 = 2 * j + 1;
  uint32_t o1 = piece_offset(P, f1 / P.Cw, f1 % P.Cw), lbo = 16u;   // lone piece: any in-bounds
  *swap = false;                                                    // partner, its weights are 0
  if (f2 < P.row_words) {
    uint32_t o2 = piece_offset(P, f2 / P.Cw, f2 % P.Cw);
    if (o2 < o1) { const uint32_t o = o1; o1 = o2; o2 = o; *swap = true; }
    lbo = o2 - o1;
  }
  return (o1 >> 4) | ((lbo >> 4) << 16);
}

// Exact n / d for n < 2^31: q = (n * m) >> (31 + s) with m = ceil(2^(31+s) / d), s = ceil(log2 d).
__device__ __forceinline__ uint32_t fast_div(uint32_t n, uint32_t m, int s) {
  return (uint32_t)(((uint64_t)n * m) >> (31 + s));
}

// Resident schedule: which pixel tiles a CTA (a pair) takes.  The U units of the grid are
// split into one group per filter slab (so a CTA expands one slab, once); inside its group of
// G units, unit g takes tiles g, g + G, g + 2G, ... of the slab: at any moment the CTAs of a
// group write neighbouring runs of every output plane, so the lines that leave the L2
// together lie together in memory (measured on 27x27 planes: 3.9 TB/s of stores against
// 2.85 TB/s when every CTA owns a contiguous range of tiles).
struct ResSched {
  uint32_t ntiles, nslabs;
  uint32_t slab, g, G;           // this unit's slab, its index in the slab's group, the group's size
  __device__ __forceinline__ uint32_t first(uint32_t s) const { return g; }
  __device__ __forceinline__ uint32_t step() const { return G; }
  __device__ __forceinline__ uint32_t count(uint32_t s) const {
    return (s == slab && g < ntiles) ? (ntiles - g + G - 1u) / G : 0u;
  }
  __device__ __forceinline__ uint32_t total() const { return count(slab); }
  // the seq-th item of the unit (seq < total()): its slab and tile
  __device__ __forceinline__ void item(uint32_t seq, uint32_t &sl, uint32_t &tile) const {
    sl = slab;
    tile = g + seq * G;
  }
};

__device__ __forceinline__ ResSched res_sched(int ntiles, int nslabs, bool pair) {
  ResSched R;
  const uint32_t unit = pair ? blockIdx.x >> 1 : blockIdx.x;
  const uint32_t units = pair ? gridDim.x >> 1 : gridDim.x;    // >= nslabs (host)
  R.ntiles = (uint32_t)ntiles;
  R.nslabs = (uint32_t)nslabs;
  // group s = units [s U / nslabs, (s + 1) U / nslabs)
  R.slab = unit * R.nslabs / units;
  while ((R.slab + 1u) * units / R.nslabs <= unit) ++R.slab;
  while (R.slab * units / R.nslabs > unit) --R.slab;
  const uint32_t g0 = R.slab * units / R.nslabs;
  R.g = unit - g0;
  R.G = (R.slab + 1u) * units / R.nslabs - g0;
  return R;
}

struct Smem {
  uint32_t wfull, wempty, pfull, pempty, afull, aempty, rawfull, rawdone;   // shared-space addresses of barrier arrays
  uint32_t *tmem_slot;
  volatile int *abort_flag;
  uint32_t ring, patch, raw;                              // shared-space byte addresses
  uint32_t alpha, nscale, nshift;                         // staged per-filter vectors
  uint32_t rank;                                          // CTA rank in its pair (0 = issues the MMAs)
};

__device__ __forceinline__ Smem carve(uint8_t *smem, const TcParams &P) {
  Smem s;
  const uint32_t base = smem_u32(smem);
  s.wfull = base;
  s.wempty = s.wfull + 8u * kMaxBarStages;
  s.pfull = s.wempty + 8u * kMaxBarStages;
  s.pempty = s.pfull + 8u * kMaxPatchBufs;
  s.afull = s.pempty + 8u * kMaxPatchBufs;
  s.aempty = s.afull + 8u * kMaxAcc;
  s.rawfull = s.aempty + 8u * kMaxAcc;
  s.rawdone = s.rawfull + 8u * kMaxRaw;
  s.tmem_slot = reinterpret_cast<uint32_t *>(
      smem + 8 * (2 * kMaxBarStages + 2 * kMaxPatchBufs + 2 * kMaxAcc + 2 * kMaxRaw));
  s.abort_flag = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
  s.ring = base + P.off_ring;
  s.patch = base + P.off_patch;
  s.raw = base + P.off_raw;
  s.alpha = base + P.off_vec;
  s.nscale = s.alpha + 4u * (uint32_t)P.vec_len;
  s.nshift = s.nscale + 4u * (uint32_t)P.vec_len;
  s.rank = P.pair ? cluster_ctarank() : 0u;
  return s;
}

// ------------------------------------------------------------------ MMA issuer (one thread)
// The MMAs of one full weight stage, unrolled.
template <int MPS, bool kPair>
__device__ __forceinline__ void issue_stage(const TcParams &P, int j0, uint32_t d_tmem,
                                            uint32_t patch_lo, uint32_t a_hi, uint32_t b_lo,
                                            uint32_t b_hi, uint32_t b_step, uint32_t tmem_sf,
                                            uint32_t first) {
#pragma unroll
  for (int jj = 0; jj < MPS; ++jj)
    umma_issue<kPair>(d_tmem, P.adesc_lo[j0 + jj] + patch_lo, a_hi, b_lo + (uint32_t)jj * b_step,
                      b_hi, P.idesc, tmem_sf, jj == 0 ? first : 1u);
}

// All MMAs of an item whose filter rows are already in shared memory (resident schedule, every
// item but the first).  The stages of the ring are contiguous, so K-step j reads its filter
// rows at b_lo0 + j b_step.  The patch descriptors of a batch of K-steps are fetched together
// and the batch is issued in straight-line code: per MMA two additions and the instruction,
// no load on its path (the stage-by-stage loop below needs ~100 cycles per MMA next to the
// other roles, the tensor core 64).
template <bool kPair>
__device__ __forceinline__ void issue_item_flat(const TcParams &P, uint32_t d_tmem, uint32_t patch_lo,
                                                uint32_t desc_hi, uint32_t b_lo0, uint32_t b_step,
                                                uint32_t tmem_sf) {
  constexpr int kBatch = 16;
  uint32_t b = b_lo0;
  for (int j0 = 0; j0 < P.nsteps; j0 += kBatch) {
    uint32_t a[kBatch];
#pragma unroll
    for (int i = 0; i < kBatch; ++i) a[i] = j0 + i < P.nsteps ? P.adesc_lo[j0 + i] + patch_lo : 0u;
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      if (j0 + i < P.nsteps) {
        umma_issue<kPair>(d_tmem, a[i], desc_hi, b, desc_hi, P.idesc, tmem_sf, (j0 + i) > 0 ? 1u : 0u);
        b += b_step;
      }
    }
  }
}

// kRes: resident schedule.  The stage barriers are then waited for only before the first item
// (the CTA stays on one slab, which stays in shared memory) and never released.
template <bool kRes, bool kPair>
__device__ void mma_loop(const TcParams &P, const Smem &S, long long i0, long long i1,
                         uint32_t tmem_base) {
  const uint32_t tmem_sf = tmem_base + (uint32_t)kSfCol;
  const int nst = (P.nsteps + P.mps - 1) / P.mps;
  const uint32_t b_lbo = (uint32_t)P.NTh * 16u;
  // descriptor halves: high word = stride between 8-row groups (128 B) and the version bit
  const uint32_t desc_hi = (128u >> 4) | (1u << 14);
  const uint32_t b_lo0 = ((S.ring & 0x3FFFFu) >> 4) | ((b_lbo >> 4) << 16);   // stage 0, K-step 0
  const uint32_t b_step = (2u * b_lbo) >> 4;                                   // next K-step
  const uint32_t stage_step = P.stage_bytes >> 4;
  int ws = 0, pb = 0, ab = 0;
  uint32_t wph = 0, pph = 0;
  uint32_t aph = 1u;                     // parity to wait for on the accumulator's empty barrier
  // streaming: items [i0, i1), item = tile * nslabs + slab; resident: the unit's own tiles of
  // its slab (see ResSched), one patch per item
  const ResSched R = res_sched(P.ntiles, P.nslabs, kPair);
  int slab = kRes ? 0 : (int)(i0 % P.nslabs);
  bool ok = true, new_tile = true;
  uint32_t patch_lo = 0;                 // patch address in descriptor units
  const uint32_t nitems = kRes ? R.total() : (uint32_t)(i1 - i0);
  for (uint32_t it = 0; it < nitems && ok; ++it) {
    if (new_tile) {
      ok = mbar_wait(S.pfull + 8u * pb, pph, S.abort_flag, &g_status_tc);
      if (!ok) break;
      patch_lo = ((S.patch + (uint32_t)pb * P.patch_bytes) & 0x3FFFFu) >> 4;
    }
    const bool wait_stages = !kRes || it == 0;
    ok = mbar_wait(S.aempty + 8u * ab, aph, S.abort_flag, &g_status_tc);
    if (!ok) break;
    tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)(ab * P.NT);
    if (kRes) ws = 0;
    if (kRes && !wait_stages) issue_item_flat<kPair>(P, d_tmem, patch_lo, desc_hi, b_lo0, b_step, tmem_sf);
    else
    for (int st = 0; st < nst && ok; ++st) {
      const int j0 = st * P.mps;
      const int nj = min(P.mps, P.nsteps - j0);
      const uint32_t b_lo = b_lo0 + (uint32_t)ws * stage_step;
      const uint32_t first = st == 0 ? 0u : 1u;     // the first MMA of an item overwrites
      if (wait_stages) {
        ok = mbar_wait(S.wfull + 8u * ws, wph, S.abort_flag, &g_status_tc);
        if (!ok) break;
        tc_fence_after();
      }
      if (nj == 4) issue_stage<4, kPair>(P, j0, d_tmem, patch_lo, desc_hi, b_lo, desc_hi, b_step, tmem_sf, first);
      else if (nj == 2) issue_stage<2, kPair>(P, j0, d_tmem, patch_lo, desc_hi, b_lo, desc_hi, b_step, tmem_sf, first);
      else if (nj == 8) issue_stage<8, kPair>(P, j0, d_tmem, patch_lo, desc_hi, b_lo, desc_hi, b_step, tmem_sf, first);
      else {
        for (int jj = 0; jj < nj; ++jj)
          umma_issue<kPair>(d_tmem, P.adesc_lo[j0 + jj] + patch_lo, desc_hi,
                            b_lo + (uint32_t)jj * b_step, desc_hi, P.idesc, tmem_sf,
                            jj == 0 ? first : 1u);
      }
      if (!kRes) umma_commit_to<kPair>(S.wempty + 8u * ws);
      if (++ws == P.stages) { ws = 0; if (!kRes) wph ^= 1u; }
    }
    if (!ok) break;
    if (kRes) {
      // every item has its own patch
      umma_commit_to<kPair>(S.afull + 8u * ab);
      umma_commit_to<kPair>(S.pempty + 8u * pb);
      if (++pb == P.npb) { pb = 0; pph ^= 1u; }
    } else {
      // next item: same tile (next slab) or the next tile
      new_tile = false;
      if (++slab == P.nslabs) { slab = 0; new_tile = true; }
      umma_commit_to<kPair>(S.afull + 8u * ab);
      if (new_tile || it + 1 == nitems) umma_commit_to<kPair>(S.pempty + 8u * pb);
      if (new_tile) { if (++pb == P.npb) { pb = 0; pph ^= 1u; } }
    }
    if (++ab == P.nacc) { ab = 0; aph ^= 1u; }
  }
}

template <bool kRes, bool kPair>
__device__ __forceinline__ void mma_role(const TcParams &P, const Smem &S, long long i0, long long i1,
                                         uint32_t tmem_base) {
  if (elect_one()) mma_loop<kRes, kPair>(P, S, i0, i1, tmem_base);
  __syncwarp();
}

// ------------------------------------------------------------------ weight producers (8 warps)
// A stage holds mps K-steps of NT filter rows: plane (2 jj + piece) of NT x 16 bytes.  K-step
// j consumes words 2j, 2j+1 of every filter row, which the word-pair-major weight layout
// keeps contiguous over the filters: a warp reads 32 rows of one K-step as one 256-byte run.
// Thread mapping: row = wt % rows_mod, and the 256 / rows_mod thread groups split the
// stage's K-steps, gs = grp_steps each (unit u of a thread = K-step grp * gs + u of the stage).
// The packed words of kPrefetch stages are in flight in registers.
constexpr int kPrefetch = 3;

struct WCursor {
  long long item;
  int st, slab;
};

// kUnits = grp_steps: K-steps a thread expands per stage.  kSwap: some K-step has its two
// pieces in descending address order (odd Cw or stride 2); otherwise the swap test is compiled
// out.  The common stage (all its K-steps exist, none is the row's lone last word) takes a
// path without per-step predicates.
// The role fills the stages of `nitems` consecutive items, the first of slab `slab0` (the
// slabs then follow cyclically), waiting for the empty barriers with parity `wph0` on the
// first round.  Streaming: all items of the CTA in one call.  Resident: one call per slab
// visit with nitems = 1 (the ring then has one stage per stage of the slab).
template <int kUnits, bool kSwap>
__device__ bool weight_role(const TcParams &P, const Smem &S, long long nitems, int slab0,
                            uint32_t wph0, int wt, int lane) {
  const long long i0 = 0, i1 = nitems;
  const int nst = (P.nsteps + P.mps - 1) / P.mps;
  const int row = wt % P.rows_mod, grp = wt / P.rows_mod;
  constexpr int gs = kUnits;
  const bool grp_on = grp * gs < P.mps && row < P.NTh;
  const uint32_t b_lbo = (uint32_t)P.NTh * 16u;
  const int row_co = (int)S.rank * P.NTh + row;          // this thread's filter inside a slab
  const int jj0 = grp * gs;                         // first K-step of this thread inside a stage
  const int nplain = (P.row_words >> 1);            // K-steps j < nplain have both words
  WCursor fc{i0, 0, slab0}, cc{i0, 0, slab0};
  auto advance = [&](WCursor &c) {
    if (++c.st == nst) { c.st = 0; ++c.item; if (++c.slab == P.nslabs) c.slab = 0; }
  };
  const uint2 *wp2 = reinterpret_cast<const uint2 *>(P.wp);
  uint2 pf[kPrefetch][kUnits];
  auto fetch = [&](uint2 dst[kUnits], const WCursor &c) {
    const int co = c.slab * P.NT + row_co;
    const bool on = grp_on && c.item < i1 && co < P.Co;
    const int j0 = c.st * P.mps + jj0;
    if (on && j0 + gs <= P.nsteps) {
      const uint2 *src = wp2 + ((size_t)j0 * P.Co + co);
#pragma unroll
      for (int u = 0; u < kUnits; ++u) dst[u] = __ldg(src + (size_t)u * P.Co);
    } else {
#pragma unroll
      for (int u = 0; u < kUnits; ++u)
        dst[u] = (on && j0 + u < P.nsteps) ? __ldg(wp2 + ((size_t)(j0 + u) * P.Co + co))
                                           : make_uint2(0u, 0u);
    }
  };
#pragma unroll
  for (int d = 0; d < kPrefetch; ++d) { fetch(pf[d], fc); advance(fc); }
  int ws = 0;
  uint32_t wph = wph0;        // parity to wait for on the empty barriers
  bool ok = true;
  const uint32_t row_off = (uint32_t)row * 16u + (uint32_t)(2 * jj0) * b_lbo;
  const uint32_t ring_end = S.ring + (uint32_t)P.stages * P.stage_bytes;
  (void)ring_end;
#pragma unroll 1
  while (cc.item < i1 && ok) {
    ok = mbar_wait_relaxed(S.wempty + 8u * ws, wph, S.abort_flag, &g_status_tc, XNOR_SLEEP_WGT);
    if (!ok) break;
    const uint32_t stage = S.ring + (uint32_t)ws * P.stage_bytes + row_off;
    const int co = cc.slab * P.NT + row_co;
    const int j0 = cc.st * P.mps + jj0;
    const bool on = grp_on && co < P.Co;
    if (on && j0 + gs <= nplain) {
      // plain stage: every K-step of this thread exists and has both of its words
      uint32_t sbits = 0u;                      // swap bits of K-steps j0 .. j0 + gs - 1
      if (kSwap) {
        const int wi = (j0 >> 5) & 31;
        sbits = __funnelshift_r(P.swap_mask[wi], P.swap_mask[(wi + 1) & 31], j0 & 31);
      }
#pragma unroll
      for (int u = 0; u < kUnits; ++u) {
        uint32_t v0[4], v1[4];
        expand_signs<false>(pf[0][u].x, v0);
        expand_signs<false>(pf[0][u].y, v1);
        const uint32_t a = stage + (uint32_t)(2 * u) * b_lbo;
        const uint32_t sw = (kSwap && ((sbits >> u) & 1u)) ? b_lbo : 0u;
        if (in_bounds(a >= S.ring && a + b_lbo + 16u <= ring_end, 1)) {
          sts128(a + sw, v0[0], v0[1], v0[2], v0[3]);
          sts128(a + b_lbo - sw, v1[0], v1[1], v1[2], v1[3]);
        }
      }
    } else if (on) {
#pragma unroll
      for (int u = 0; u < kUnits; ++u) {
        const int j = j0 + u;
        if (j < P.nsteps) {
          const bool swap = (P.swap_mask[(j >> 5) & 31] >> (j & 31)) & 1u;
          const uint32_t keep = j < nplain ? 0xFFFFFFFFu : 0u;   // lone last word: partner is 0
          uint32_t v0[4], v1[4];
          expand_signs<false>(pf[0][u].x, v0);
          expand_signs<false>(pf[0][u].y, v1);
          v1[0] &= keep; v1[1] &= keep; v1[2] &= keep; v1[3] &= keep;
          const uint32_t a = stage + (uint32_t)(2 * u) * b_lbo;
          if (in_bounds(a >= S.ring && a + b_lbo + 16u <= ring_end, 2)) {
            sts128(swap ? a + b_lbo : a, v0[0], v0[1], v0[2], v0[3]);
            sts128(swap ? a : a + b_lbo, v1[0], v1[1], v1[2], v1[3]);
          }
        }
      }
    }
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) { if (P.pair) mbar_arrive_cluster(S.wfull + 8u * ws, 0u); else mbar_arrive(S.wfull + 8u * ws); }
    if (++ws == P.stages) { ws = 0; wph ^= 1u; }
    advance(cc);
    // the queue of packed words moves up one stage; the freed slot is refilled
#pragma unroll
    for (int d = 0; d + 1 < kPrefetch; ++d)
#pragma unroll
      for (int u = 0; u < kUnits; ++u) pf[d][u] = pf[d + 1][u];
    fetch(pf[kPrefetch - 1], fc);
    advance(fc);
  }
  return ok;
}

template <int kUnits>
__device__ __forceinline__ bool weight_role_swap(const TcParams &P, const Smem &S,
                                                 long long nitems, int slab0, uint32_t wph0,
                                                 int wt, int lane) {
  return P.any_swap ? weight_role<kUnits, true>(P, S, nitems, slab0, wph0, wt, lane)
                    : weight_role<kUnits, false>(P, S, nitems, slab0, wph0, wt, lane);
}

__device__ __forceinline__ bool weight_dispatch(const TcParams &P, const Smem &S, long long nitems,
                                                int slab0, uint32_t wph0, int wt, int lane) {
  if (P.grp_steps == 4) return weight_role_swap<4>(P, S, nitems, slab0, wph0, wt, lane);
  if (P.grp_steps == 2) return weight_role_swap<2>(P, S, nitems, slab0, wph0, wt, lane);
  return weight_role_swap<1>(P, S, nitems, slab0, wph0, wt, lane);
}

// ------------------------------------------------------------------ patch producers
// A group of P.pat_group warps (the three patch warps) builds the CTA's patches one after the
// other, all warps on the same patch: units of (32 stream positions, phase plane, up to 4 channel words) are dealt round
// robin.  The packed pixels a patch touches are ONE contiguous range of x_packed: input rows
// g0 .. g1 - 1 of the N*H rows (images follow one another in memory, the zero rows and
// columns of the stream exist only in the patch).  Every patch buffer has a raw buffer; the
// group's first warp brings a patch's range into it with one bulk copy (an aligned superset
// inside the tensor; the ragged last words of the tensor, if any, by plain loads) as soon as
// the group is done with the buffer's previous patch, so the rows of the next patches are on
// their way while one is expanded.  Padding and the channel tail become the value 0 through
// masks folded into the sign mask and the magnitude constants.
// Streaming: one patch per tile of the CTA's range.  Resident (kRes): one patch per item.
template <bool kRes>
__device__ void patch_role(const TcParams &P, const Smem &S, long long i0, long long i1, int pw,
                           int lane) {
  const ResSched R = res_sched(P.ntiles, P.nslabs, P.pair != 0);
  const int tile0 = kRes ? 0 : (int)(i0 / P.nslabs);
  const uint32_t npatches = kRes ? R.total()
                                 : (uint32_t)((i1 - 1) / P.nslabs) - (uint32_t)tile0 + 1u;
  const int s = P.stride, phases = s * s;
  const uint32_t plane_bytes = (uint32_t)P.ppix * 16u;
  const bool vec = (P.Cw & 3) == 0;
  // nibble masks of the channel tail, one per expanded register
  uint32_t tm[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) tm[r] = ((P.tail_mask >> r) & 0x11111111u) * 0xFu;
  const bool tail = P.tail_mask != 0xFFFFFFFFu;
  const uint32_t row_bytes = (uint32_t)P.W * (uint32_t)P.Cw * 4u;
  const size_t tensor_bytes = (size_t)P.N * P.H * row_bytes;
  // pairs: work tile t is stream tiles 2t (rank 0) and 2t + 1 (rank 1)
  const uint32_t tmul = P.pair ? 2u : 1u;
  const int ngrp = (P.Cw + 3) >> 2;                       // groups of 4 channel words
  const int npass = (P.ppix + 31) >> 5;
  const int nunits = npass * phases * ngrp;

  auto tile_of = [&](uint32_t seq) {
    if (!kRes) return tile0 + (int)seq;
    uint32_t sl, t;
    R.item(seq, sl, t);
    return (int)t;
  };
  // input rows [g0, g1) (of the N*H rows of the tensor) that the patch of a tile reads
  auto row_range = [&](int tile, int &g0, int &g1) {
    const uint32_t m0 = ((uint32_t)tile * tmul + S.rank) * kTileM;
    const uint32_t mlast = min(m0 + (uint32_t)P.ppix - 1u, (uint32_t)P.L - 1u);
    const uint32_t r0 = fast_div(m0, P.div_wq_m, P.div_wq_s);
    const uint32_t r1 = fast_div(mlast, P.div_wq_m, P.div_wq_s);
    const uint32_t n0 = fast_div(r0, P.div_hq_m, P.div_hq_s);
    const uint32_t n1 = fast_div(r1, P.div_hq_m, P.div_hq_s);
    const int ry0 = (int)(r0 - n0 * (uint32_t)P.Hq), ry1 = (int)(r1 - n1 * (uint32_t)P.Hq);
    const int t0 = min(max((ry0 - P.leadY) * s, 0), P.H);
    const int t1 = min(max((ry1 - P.leadY) * s + s, 0), P.H);
    g0 = (int)n0 * P.H + t0;
    g1 = (int)n1 * P.H + t1;
  };
  // a subgroup's first warp, lane 0: starts the copy of a patch's rows into raw buffer rb
  auto start_copy = [&](uint32_t seq, uint32_t rb) {
    int g0, g1;
    row_range(tile_of(seq), g0, g1);
    const uint32_t bar = S.rawfull + 8u * rb;
    const uint32_t dst = S.raw + rb * P.raw_bytes;
    if (g1 <= g0) { mbar_arrive(bar); return; }          // nothing but padding
    const size_t b0 = (size_t)g0 * row_bytes, b1 = (size_t)g1 * row_bytes;
    const size_t a0 = b0 & ~(size_t)15;
    const size_t a1 = min((b1 + 15) & ~(size_t)15, tensor_bytes & ~(size_t)15);
    const uint32_t bulk = a1 > a0 ? (uint32_t)(a1 - a0) : 0u;
    for (size_t b = a0 + bulk; b < b1; b += 4)           // at most 3 words, at the tensor's end
      if (in_bounds((uint32_t)(b - a0) + 4u <= P.raw_bytes, 3))
        sts32(dst + (uint32_t)(b - a0), __ldg(P.xp + (b >> 2)));
    if (bulk && in_bounds(bulk <= P.raw_bytes && a0 + bulk <= tensor_bytes, 4)) {
      mbar_arrive_expect_tx(bar, bulk);
      bulk_copy_g2s(dst, reinterpret_cast<const uint8_t *>(P.xp) + a0, bulk, bar);
    } else {
      mbar_arrive(bar);
    }
  };

  // The group works as `nsub` subgroups of equal size; subgroup sg builds patches sg,
  // sg + nsub, ... (nsub <= npb: a barrier's parity tells apart only two consecutive uses of
  // a buffer, so no subgroup may run more than one use ahead of the consumer).
  const uint32_t nsub = (uint32_t)P.pat_sub, gsize = (uint32_t)P.pat_group / nsub;
  const uint32_t sg = (uint32_t)pw % nsub, mi = (uint32_t)pw / nsub;
  // The subgroup's k-th patch (patch sg + k nsub of the CTA) expands from the subgroup's raw
  // buffer k % nraw; its rows are fetched as soon as the subgroup is done with patch k - nraw.
  const uint32_t nraw = (uint32_t)P.nraw, rb0 = sg * nraw;
  bool ok = true;
  uint32_t kc = 0;                           // patches of the subgroup whose copy has been started
  if (mi == 0) {
    for (; kc < nraw && sg + kc * nsub < npatches; ++kc)
      if (lane == 0) start_copy(sg + kc * nsub, rb0 + kc);
  }
  uint32_t k = 0;
#pragma unroll 1
  for (uint32_t seq = sg; seq < npatches && ok; seq += nsub, ++k) {
    const int tile = tile_of(seq);
    const uint32_t pb = seq % (uint32_t)P.npb;
    const uint32_t use = seq / (uint32_t)P.npb;
    const uint32_t rb = rb0 + k % nraw, ruse = k / nraw;
    if (mi == 0 && k >= 1u && sg + kc * nsub < npatches) {
      // kc = k - 1 + nraw: the raw buffer of patch k - 1 is free once every warp of the
      // subgroup has expanded that patch
      const uint32_t crb = rb0 + kc % nraw;
      ok = mbar_wait_relaxed(S.rawdone + 8u * crb, (kc / nraw - 1u) & 1u, S.abort_flag,
                             &g_status_tc, XNOR_SLEEP_PAT);
      if (!ok) break;
      fence_proxy_async();
      if (lane == 0) start_copy(sg + kc * nsub, crb);
      ++kc;
    }
    int g0, g1;
    row_range(tile, g0, g1);
    ok = mbar_wait_relaxed(S.rawfull + 8u * rb, ruse & 1u, S.abort_flag, &g_status_tc, XNOR_SLEEP_PAT);
    if (!ok) break;
    ok = mbar_wait_relaxed(S.pempty + 8u * pb, (use & 1u) ^ 1u, S.abort_flag, &g_status_tc,
                           XNOR_SLEEP_PAT);
    if (!ok) break;
    const uint32_t patch = S.patch + pb * P.patch_bytes;
    const uint32_t m0 = ((uint32_t)tile * tmul + S.rank) * kTileM;
    const uint32_t raw = S.raw + rb * P.raw_bytes +
                         (uint32_t)(((size_t)g0 * row_bytes) & 15u);   // where row g0 starts
    // kPatUnits units at a time: their index arithmetic and loads are independent chains the
    // warp can overlap, then all are expanded
#pragma unroll 1
    for (int u0 = (int)mi; u0 < nunits; u0 += kPatUnits * (int)gsize) {
      uint32_t src[kPatUnits], dst[kPatUnits], sm[kPatUnits], mc[kPatUnits][3], wv[kPatUnits][4];
      int w0[kPatUnits];
      bool on[kPatUnits], real[kPatUnits];
#pragma unroll
      for (int b = 0; b < kPatUnits; ++b) {
        const int u = u0 + b * (int)gsize;
        const int pass = (int)fast_div((uint32_t)u, P.div_pg_m, P.div_pg_s);
        const int rem = u - pass * (phases * ngrp);
        const int phase = (int)fast_div((uint32_t)rem, P.div_g_m, P.div_g_s);
        w0[b] = (rem - phase * ngrp) * 4;
        const int q = pass * 32 + lane;
        on[b] = u < nunits && q < P.ppix;
        const uint32_t sq = m0 + (uint32_t)q;
        const uint32_t r = fast_div(sq, P.div_wq_m, P.div_wq_s);
        const int c = (int)(sq - r * (uint32_t)P.Wq);
        const uint32_t n = fast_div(r, P.div_hq_m, P.div_hq_s);
        const int ry = (int)(r - n * (uint32_t)P.Hq);
        const int py = phase >> (s - 1), px = phase & (s - 1);     // stride 1 or 2
        const int rrow = (ry - P.leadY) * s + py, rcol = (c - P.leadX) * s + px;
        real[b] = on[b] && sq < (uint32_t)P.L && ry >= P.leadY && c >= P.leadX && rrow < P.H &&
                  rcol < P.W;
        const uint32_t keep = real[b] ? 0xFFFFFFFFu : 0u;        // padding expands to 0
        sm[b] = 0x88888888u & keep;
        mc[b][0] = 0xCCCCCCCCu & keep; mc[b][1] = 0xAAAAAAAAu & keep; mc[b][2] = 0x99999999u & keep;
        src[b] = raw + (uint32_t)((((int)n * P.H + rrow - g0) * P.W + rcol) * P.Cw + w0[b]) * 4u;
        dst[b] = patch + (uint32_t)(phase * P.Cw + w0[b]) * plane_bytes + (uint32_t)q * 16u;
      }
#pragma unroll
      for (int b = 0; b < kPatUnits; ++b) {
        wv[b][0] = wv[b][1] = wv[b][2] = wv[b][3] = 0u;
        if (real[b] && in_bounds(src[b] >= S.raw + rb * P.raw_bytes &&
                                 src[b] + 4u * (uint32_t)min(4, P.Cw - w0[b]) <= S.raw + (rb + 1u) * P.raw_bytes, 6)) {
          if (vec) {
            lds128(src[b], wv[b]);
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (w0[b] + i < P.Cw) wv[b][i] = lds32(src[b] + (uint32_t)i * 4u);
          }
        }
      }
#pragma unroll
      for (int b = 0; b < kPatUnits; ++b) {
        if (on[b]) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (w0[b] + i < P.Cw) {
              const uint32_t w = wv[b][i];
              uint32_t v0 = ((w << 3) & sm[b]) ^ mc[b][0];
              uint32_t v1 = ((w << 2) & sm[b]) ^ mc[b][1];
              uint32_t v2 = ((w << 1) & sm[b]) ^ mc[b][2];
              uint32_t v3 = (w & sm[b]) ^ mc[b][2];
              if (tail && w0[b] + i == P.Cw - 1) {       // channels beyond C_in are 0
                v0 &= tm[0]; v1 &= tm[1]; v2 &= tm[2]; v3 &= tm[3];
              }
              if (in_bounds(dst[b] + (uint32_t)i * plane_bytes >= patch &&
                            dst[b] + (uint32_t)i * plane_bytes + 16u <= patch + P.patch_bytes, 5))
                sts128(dst[b] + (uint32_t)i * plane_bytes, v0, v1, v2, v3);
            }
          }
        }
      }
    }
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      mbar_arrive(S.rawdone + 8u * rb);
      if (P.pair) mbar_arrive_cluster(S.pfull + 8u * pb, 0u); else mbar_arrive(S.pfull + 8u * pb);
    }
  }
  if (!ok && mi == 0) {
    // gave up: the copies this warp started last (one per buffer at most can still be in
    // flight) must land before the CTA's shared memory is released
    for (uint32_t back = 1; back <= nraw && back <= kc; ++back) {
      const uint32_t c = kc - back;
      for (int i = 0; i < (1 << 20) && !mbar_try(S.rawfull + 8u * (rb0 + c % nraw), (c / nraw) & 1u); ++i) {}
    }
  }
}

// ------------------------------------------------------------------ epilogue (4 warps)
// Warp w reads tensor-memory lanes 32 w .. +31 (pixels), all the slab's columns (filters).
// Lane = pixel, so for one filter a warp stores 32 consecutive stream pixels: a contiguous
// run of the NCHW output row.
// Drains `nitems` items, the k0-th and following of the CTA: streaming, items i0, i0 + 1, ...
// (item = tile * nslabs + slab); resident, tiles tile0, tile0 + tstep, ... of slab `slab0`.
// Of every item this warp takes
// the 16-column groups e, e + esplit, ... (esplit warps share a quarter of the lanes).
// kFuse: the groups a warp takes come in pairs (32 consecutive filters = one packed word of the
// next layer's input); see the fused emit below.
template <bool kRes, bool kFuse>
__device__ bool epilogue_role(const TcParams &P, const Smem &S, long long i0, int slab0, int tile0,
                              int tstep, uint32_t nitems, long long k0, uint32_t tmem_base,
                              int quarter, int e, int lane) {
  const int b_end = P.NT / 16;
  const int esplit = kRes ? P.epi_split : 1;
  // the k-th group of this warp: groups e, e + esplit, ... or, fused, the two groups of the
  // pairs e, e + esplit, ...
  const int units = kFuse ? b_end / 2 : b_end;
  const int nk = ((units - e + esplit - 1) / esplit) * (kFuse ? 2 : 1);
  auto group_of = [&](int k) {
    return kFuse ? 2 * (e + esplit * (k >> 1)) + (k & 1) : e + esplit * k;
  };
  const size_t HoWo = (size_t)P.Ho * P.Wo;
  const uint32_t howo = (uint32_t)HoWo;
  const size_t out_elems = (size_t)P.N * P.Co * HoWo;
  (void)out_elems;
  // the fast store paths: offsets of 16 consecutive filters fit 32 bits, no integer output
  const bool small = HoWo < ((size_t)1 << 27) && P.acc_out == nullptr;
  const bool relu = P.relu != 0;
  const bool plain = small && P.residual == nullptr, with_res = small && P.residual != nullptr;
  const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
  int tile, slab;
  if (kRes) { slab = slab0; tile = tile0; }
  else { tile = (int)(i0 / P.nslabs); slab = (int)(i0 - (long long)tile * P.nslabs); }
  bool ok = true;
  // this lane's output pixel in a tile: whether it exists, its K, offset of (image, filter 0, pixel)
  struct Pix { bool valid; float kv; size_t obase; size_t gpix; };   // gpix: pixel index over all images
  auto decode = [&](int t) {
    Pix px{false, 0.0f, 0, 0};
    const uint32_t m = ((uint32_t)t * (P.pair ? 2u : 1u) + S.rank) * kTileM + (uint32_t)(quarter * 32 + lane);
    if (m < (uint32_t)P.L) {
      const uint32_t r = fast_div(m, P.div_wq_m, P.div_wq_s);
      const int ox = (int)(m - r * (uint32_t)P.Wq);
      const uint32_t n = fast_div(r, P.div_hq_m, P.div_hq_s);
      const int oy = (int)(r - n * (uint32_t)P.Hq);
      if (ox < P.Wo && oy < P.Ho) {
        const size_t pix = (size_t)oy * P.Wo + ox;
        px.valid = true;
        px.kv = __ldg(P.K + (size_t)n * HoWo + pix);
        px.obase = (size_t)n * P.Co * HoWo + pix;
        px.gpix = (size_t)n * HoWo + pix;
      }
    }
    return px;
  };
  Pix px = decode(tile);
  int ab = (int)(k0 % P.nacc);            // accumulator buffer of the next item and the parity
  uint32_t fph = (uint32_t)(k0 / P.nacc) & 1u;   // of its full barrier
  for (uint32_t it = 0; it < nitems && ok; ++it) {
    const bool valid = px.valid;
    const float kv = px.kv;
    const size_t obase = px.obase;
    const size_t obase_pix = px.gpix;
    // the item after this one; its pixel is decoded (and its K loaded) while this one drains
    int ntile = tile, nslab = slab;
    bool next_new;
    if (kRes) {
      next_new = true;
      ntile += tstep;
    } else {
      next_new = false;
      if (++nslab == P.nslabs) { nslab = 0; ++ntile; next_new = true; }
    }
    if (P.residual != nullptr && e == 0) {
      // The residual tile of this item is pulled into L2 while its MMAs run: the loads in the
      // drain loop then see L2 latency only, and the bytes in flight are not bounded by registers.
      // The warp's pixels are one run of a filter's plane (at most 128 bytes: two lines), so a
      // lane takes a filter and touches the two ends of its run: a handful of instructions per
      // item instead of one prefetch per filter and lane.
      const unsigned vm = __ballot_sync(0xffffffffu, valid);
      if (vm != 0u) {
        const unsigned long long o0 = __shfl_sync(0xffffffffu, (unsigned long long)obase, __ffs(vm) - 1);
        const unsigned long long o1 = __shfl_sync(0xffffffffu, (unsigned long long)obase, 31 - __clz(vm));
        const int nf = min(P.NT, P.Co - slab * P.NT);
        const float *rp = P.residual + (size_t)(slab * P.NT) * HoWo;
        for (int j = lane; j < nf; j += 32) {
          asm volatile("prefetch.global.L2 [%0];" ::"l"(rp + o0 + (size_t)j * HoWo));
          asm volatile("prefetch.global.L2 [%0];" ::"l"(rp + o1 + (size_t)j * HoWo));
        }
      }
    }
    ok = mbar_wait_relaxed(S.afull + 8u * ab, fph, S.abort_flag, &g_status_tc, XNOR_SLEEP_EPI);
    if (!ok) break;
    tc_fence_after();
    const uint32_t t_acc = t_lane + (uint32_t)(ab * P.NT);
    const int co0 = slab * P.NT;
    Pix npx = px;
    if (next_new && it + 1 < nitems) npx = decode(ntile);

    // Store addresses step from filter to filter by one multiply-add each (forming every
    // address from the group's base takes two instructions per store and measured slower).
    auto emit = [&](int b, const int32_t r[16]) {
      if (!valid) return;
      const int co = co0 + b * 16;
      float *op = P.out + obase + (size_t)co * HoWo;
      if (co + 16 <= P.Co && plain) {
        float4 al[4];
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4)
          al[j4] = lds_f4(S.alpha + (uint32_t)(co * 4 + j4 * 16));
        // the 16 products first, then the 16 stores (and the ReLU test once per group, not per
        // value): two multiplies, an address and a store per output
        float v[16];
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4) {
          v[j4 * 4 + 0] = __fmul_rn(__fmul_rn(__int_as_float(r[j4 * 4 + 0]), kv), al[j4].x);
          v[j4 * 4 + 1] = __fmul_rn(__fmul_rn(__int_as_float(r[j4 * 4 + 1]), kv), al[j4].y);
          v[j4 * 4 + 2] = __fmul_rn(__fmul_rn(__int_as_float(r[j4 * 4 + 2]), kv), al[j4].z);
          v[j4 * 4 + 3] = __fmul_rn(__fmul_rn(__int_as_float(r[j4 * 4 + 3]), kv), al[j4].w);
        }
        if (relu) {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = fmaxf(v[j], 0.0f);
        }
        // one address per store, each one multiply-add from the one before; streaming stores
        // (the output is not read again by this kernel: evict-first keeps the L2 for the inputs;
        // 6-8 % on the ResNet layers run back to back, nothing on a whole step)
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          if (in_bounds(obase + (size_t)(co + j) * HoWo < out_elems, 7)) __stcs(op, v[j]);
          op += howo;
        }
      } else if (co + 16 <= P.Co && with_res) {
        const float *rp = P.residual + obase + (size_t)co * HoWo;
        float res[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) { res[j] = *rp; rp += howo; }
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4) {
          const float4 al = lds_f4(S.alpha + (uint32_t)(co * 4 + j4 * 16));
          const float a4[4] = {al.x, al.y, al.z, al.w};
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const float v = __fmul_rn(__fmul_rn(__int_as_float(r[j4 * 4 + jj]), kv), a4[jj]) + res[j4 * 4 + jj];
            if (in_bounds((size_t)(op - P.out) < out_elems, 8)) __stcs(op, relu ? fmaxf(v, 0.0f) : v);
            op += howo;
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
            float v = __fmul_rn(__fmul_rn(d, kv), lds_f(S.alpha + (uint32_t)((co + j) * 4)));
            if (P.residual) v += res[j];
            if (relu) v = fmaxf(v, 0.0f);
            if (in_bounds(o0 + (size_t)j * HoWo < out_elems, 9)) P.out[o0 + (size_t)j * HoWo] = v;
            if (P.acc_out) {
              int32_t *ap = P.acc_out + o0 + (size_t)j * HoWo;
              *ap = (P.acc_accum ? *ap : 0) + (__float2int_rn(d) << P.acc_shift);
            }
          }
        }
      }
    };

    // Fused: out = D K alpha (+ residual) as above (stored only if the caller wants the fp32
    // tensor), then y = fmaf(scale, out, shift) of the next layer's BatchNorm, the sign bit of
    // y into the word of this pair of groups, |y| into this warp's partial sum for A.
    uint32_t word = 0u;
    float as0 = 0.0f, as1 = 0.0f, as2 = 0.0f, as3 = 0.0f;     // four chains of the |y| sum
    auto emit_fused = [&](int b, const int32_t r[16]) {
      if (!valid) return;
      const int co = co0 + b * 16;
      uint32_t half = 0u;                     // the 16 sign bits of this group
      float *op = P.out + obase + (size_t)co * HoWo;
      float res[16];                          // all 16 residual loads in flight together
      if (P.residual != nullptr) {
        const float *rp = P.residual + obase + (size_t)co * HoWo;
#pragma unroll
        for (int j = 0; j < 16; ++j) { res[j] = *rp; rp += howo; }
      }
#pragma unroll
      for (int j4 = 0; j4 < 4; ++j4) {
        const float4 al = lds_f4(S.alpha + (uint32_t)(co * 4 + j4 * 16));
        float4 sc = make_float4(1.0f, 1.0f, 1.0f, 1.0f), sh = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (P.nscale != nullptr) {
          sc = lds_f4(S.nscale + (uint32_t)(co * 4 + j4 * 16));
          sh = lds_f4(S.nshift + (uint32_t)(co * 4 + j4 * 16));
        }
        const float a4[4] = {al.x, al.y, al.z, al.w};
        const float s4[4] = {sc.x, sc.y, sc.z, sc.w}, h4[4] = {sh.x, sh.y, sh.z, sh.w};
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int j = j4 * 4 + jj;
          float v = __fmul_rn(__fmul_rn(__int_as_float(r[j]), kv), a4[jj]);
          if (P.residual != nullptr) v += res[j];
          if (relu) v = fmaxf(v, 0.0f);
          if (P.out != nullptr && in_bounds(obase + (size_t)(co + j) * HoWo < out_elems, 10)) *op = v;
          op += howo;
          const float y = P.nscale != nullptr ? __fmaf_rn(s4[jj], v, h4[jj]) : v;
          half |= (y >= 0.0f ? 1u : 0u) << j;
          if (jj == 0) as0 += fabsf(y);
          else if (jj == 1) as1 += fabsf(y);
          else if (jj == 2) as2 += fabsf(y);
          else as3 += fabsf(y);
        }
      }
      word |= half << (co & 16);              // C_out % 32 == 0: a group is the low or the high half
    };

    // 16 columns at a time: load, wait, scale and store.  (Loading the next 16 during the
    // stores of the current ones saves the ~50 cycles of a tensor-memory load per group but
    // costs 16 register copies, which take longer here.)
    int32_t cur[16];
#pragma unroll 1
    for (int k = 0; k < nk; ++k) {
      const int b = group_of(k);
      tmem_ld16(t_acc + (uint32_t)(b * 16), cur);
      tmem_wait16(cur);
      if (k + 1 == nk) {                         // that was the last load: release the buffer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) { if (P.pair) mbar_arrive_cluster(S.aempty + 8u * ab, 0u); else mbar_arrive(S.aempty + 8u * ab); }
      }
      if (kFuse) {
        // C_out is a multiple of 32, so a pair of groups lies inside the filters or (last slab)
        // wholly beyond them
        if (co0 + b * 16 >= P.Co) continue;
        emit_fused(b, cur);
        if ((k & 1) && valid) {                  // the pair is complete: its word of the next input
          if (in_bounds(obase_pix < (size_t)P.N * HoWo && ((co0 + b * 16) >> 5) < P.Cw_next, 11))
            P.xp_next[(obase_pix) * (size_t)P.Cw_next + (size_t)((co0 + b * 16) >> 5)] = word;
          word = 0u;
        }
      } else {
        emit(b, cur);
      }
    }
    if (kFuse && valid && in_bounds(obase_pix < (size_t)P.N * HoWo, 12))
      P.A_part[(size_t)(slab * esplit + e) * ((size_t)P.N * HoWo) + obase_pix] = (as0 + as1) + (as2 + as3);
    px = npx;
    tile = ntile;
    slab = nslab;
    if (++ab == P.nacc) { ab = 0; fph ^= 1u; }
  }
  return ok;
}

template <bool kRes, bool kPair, bool kFuse>
__global__ void __launch_bounds__(kThreads, 1)
binconv_tc_kernel(const __grid_constant__ TcParams P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Smem S = carve(smem, P);

  if (tid == 0) {
    // In a pair the producers of both CTAs arrive on the barriers of rank 0 (whose MMA warp
    // waits for them); the MMA warp's commits reach the consumer barriers of both CTAs.
    constexpr uint32_t kCtas = kPair ? 2u : 1u;
    for (int i = 0; i < kMaxBarStages; ++i) {
      mbar_init(S.wfull + 8u * i, (uint32_t)P.wgt_warps * kCtas);
      mbar_init(S.wempty + 8u * i, 1);
    }
    for (int i = 0; i < kMaxPatchBufs; ++i) {
      mbar_init(S.pfull + 8u * i, (uint32_t)(P.pat_group / P.pat_sub) * kCtas);
      mbar_init(S.pempty + 8u * i, 1);
    }
    for (int i = 0; i < kMaxRaw; ++i) {
      mbar_init(S.rawfull + 8u * i, 1);
      mbar_init(S.rawdone + 8u * i, (uint32_t)(P.pat_group / P.pat_sub));
    }
    for (int i = 0; i < kMaxAcc; ++i) {
      mbar_init(S.afull + 8u * i, 1);
      mbar_init(S.aempty + 8u * i, (kRes ? kEpiWarps * P.epi_split : kEpiWarps) * kCtas);
    }
    *S.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // per-filter vectors of the epilogue, zero beyond C_out (one global round trip per CTA
  // instead of one per 16 columns drained); alpha carries the call's extra output factor
  // (1 except in the passes of a k-bit convolution; a product with 1 is exact)
  for (int i = tid; i < P.vec_len; i += kThreads) {
    reinterpret_cast<float *>(smem + P.off_vec)[i] = i < P.Co ? __fmul_rn(__ldg(P.alpha + i), P.out_scale) : 0.0f;
    if (kFuse && P.nscale != nullptr) {
      reinterpret_cast<float *>(smem + P.off_vec)[P.vec_len + i] = i < P.Co ? __ldg(P.nscale + i) : 0.0f;
      reinterpret_cast<float *>(smem + P.off_vec)[2 * P.vec_len + i] = i < P.Co ? __ldg(P.nshift + i) : 0.0f;
    }
  }
  if (warp == kMmaWarp) {
    if (kPair) {
      // the same warp of both CTAs of the pair allocates, at the same shared-memory offset
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(S.tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(S.tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
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
  // no CTA of a pair signals a barrier of the other before that one has set it up
  if (kPair) cluster_sync();

  // this CTA's (pair's) contiguous range of work items; item = tile * nslabs + slab
  // (streaming) or slab * ntiles + tile (resident); for a pair a tile is two stream tiles
  const long long total = (long long)P.ntiles * P.nslabs;
  const unsigned unit = kPair ? blockIdx.x >> 1 : blockIdx.x, units = kPair ? gridDim.x >> 1 : gridDim.x;
  const long long i0 = total * unit / units;
  const long long i1 = total * (unit + 1) / units;
  const ResSched R = res_sched(P.ntiles, P.nslabs, kPair);
  if (kRes ? R.total() > 0u : i0 < i1) {
    const int wt = tid - 32 * kWgtWarp0;
    if (warp == kMmaWarp) { if (S.rank == 0) mma_role<kRes, kPair>(P, S, i0, i1, tmem_base); }
    else if (warp >= kPatWarp0) patch_role<kRes>(P, S, i0, i1, warp - kPatWarp0, lane);
    else if (!kRes) {
      if (warp < kEpiWarps)
        epilogue_role<false, kFuse>(P, S, i0, 0, 0, 0, (uint32_t)(i1 - i0), 0, tmem_base, warp, 0, lane);
      else weight_dispatch(P, S, i1 - i0, (int)(i0 % P.nslabs), 1u, wt, lane);
    } else {
      // Slab visits of this CTA in order.  The weight warps expand the slab, then every
      // worker warp drains its share of the visit's items.
      const bool wgt = warp >= kWgtWarp0;
      const int e = wgt ? 1 + (warp - kWgtWarp0) / 4 : 0;
      uint32_t visit = 0, done = 0;
      bool ok = true;
      for (uint32_t slab = 0; slab < R.nslabs && ok; ++slab) {
        const uint32_t n = R.count(slab);
        if (n == 0u) continue;
        if (wgt) ok = weight_dispatch(P, S, 1, (int)slab, (visit & 1u) ^ 1u, wt, lane);
        if (ok && e < P.epi_split)
          ok = epilogue_role<true, kFuse>(P, S, 0, (int)slab, (int)R.first(slab), (int)R.step(), n,
                                          done, tmem_base, warp & 3, e, lane);
        done += n;
        ++visit;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  // both CTAs of a pair are done with each other's barriers and tensor memory
  if (kPair) cluster_sync();
  if (warp == kMmaWarp) {
    if (kPair)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                   ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    else
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

// Weight-thread mapping and stage size for slabs of NT filters: rows_mod threads cover the
// rows of a K-step, the other thread groups take other K-steps of the stage; a stage is up to
// 32 KB of expanded weights.
void plan_stage(TcParams &P) {
  int ntp = 16;
  while (ntp < P.NTh) ntp *= 2;                         // 16 .. 256
  P.rows_mod = ntp;
  const int groups = std::max(1, 32 * P.wgt_warps / P.rows_mod);   // 1 .. 16
  P.mps = std::max(2, std::min(8, 1024 / ntp));
  while (P.mps > 4 && P.nsteps < 3 * P.mps) P.mps /= 2;   // short items: smaller stages start sooner
  if (P.mps > 4 * groups) P.mps = 4 * groups;           // a thread expands at most 4 K-steps of a stage
  P.grp_steps = std::max(1, P.mps / groups);            // 4, 4, 2, 1, 1
  P.stage_bytes = (uint32_t)P.mps * (uint32_t)P.NTh * 32u;
}

// Filters per slab for `ns` slabs.  A pair splits the rows of a slab between its two CTAs
// (halves of a multiple of 16 rows each).
int slab_width(int Co, int ns, bool pair) {     // pair: also set for the fused epilogue (32-filter words)
  const int q = pair ? 32 : 16;
  return ((Co + ns - 1) / ns + q - 1) / q * q;
}

// schedule: 0 = resident when the slab fits, 1 = streaming.  pair: CTA pairs (clusters of 2).
Plan make_plan(const ConvGeom &g, int schedule, bool pair, bool fuse = false) {
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
  P.ntiles = (int)((P.L + kTileM - 1) / kTileM);
  P.pair = pair ? 1 : 0;
  if (pair) P.ntiles = (P.ntiles + 1) / 2;               // a work tile is two stream tiles
  const int halo = (dymax - P.dymin) * P.Wq + (dxmax - P.dxmin);
  P.ppix = (kTileM + halo + 1 + 7) / 8 * 8;             // +1: a lone piece reads one pixel further
  if (P.L + P.ppix + 2 * kTileM >= (1ll << 31)) return pl;  // stream positions stay below 2^31
  // packed input rows one patch can touch: its stream rows, `stride` input rows each; the
  // copy is an aligned superset (up to 12 bytes before, 15 after)
  const long long raw_rows = ((long long)(P.ppix - 1) / P.Wq + 2) * s;
  const long long raw_bytes = (raw_rows * g.W * g.Cw * 4 + 12 + 15 + 15) / 16 * 16;
  if (raw_bytes > (long long)kSmemMax) return pl;
  P.raw_bytes = (uint32_t)raw_bytes;
  P.nplanes = s * s * g.Cw;
  P.patch_bytes = (uint32_t)P.nplanes * (uint32_t)P.ppix * 16u;
  // K-steps
  P.row_words = g.kh * g.kw * g.Cw;
  P.nsteps = (P.row_words + 1) / 2;
  if (P.nsteps > kMaxSteps) return pl;
  // shared memory: control, weight stages, patch buffers
  // per-filter vectors (alpha; fused: also the next scale and shift), padded to whole slabs
  P.off_vec = (uint32_t)((kCtrlBytes + 127) / 128 * 128);
  P.vec_len = (g.Co + 15) / 16 * 16 + 512;          // every slab of any width ends inside it
  P.off_ring = (uint32_t)((P.off_vec + (size_t)(fuse ? 3 : 1) * P.vec_len * 4 + 127) / 128 * 128);
  if (P.off_ring + 4096 > kSmemMax) return pl;
  const size_t avail = kSmemMax - P.off_ring;
  // st weight stages, pb patch buffers, nraw raw buffers for each subgroup of patch warps
  auto subgroups = [&](int pb) { return (P.pat_group == kPatWarps && pb >= kPatWarps) ? kPatWarps : 1; };
  auto fits = [&](int st, int pb, int nraw) {
    return (size_t)st * P.stage_bytes + (size_t)pb * P.patch_bytes +
           (size_t)(subgroups(pb) * nraw) * P.raw_bytes <= avail;
  };
  P.wgt_warps = kWgtWarps;
  P.pat_group = kPatWarps;
  // as few slabs as fit two accumulators in the tensor-memory columns
  const int max_nt = pair ? 224 : 240;
  const int min_slabs = (g.Co + max_nt - 1) / max_nt;
  int stages = 0, npb = 0;
  P.resident = 0;
  if (schedule == 0) {
    // Resident: the widest slab whose expanded rows fit beside two patches.  Every slab
    // needs its own patch per tile and narrow MMAs re-read the pixel operand more often, so
    // (measured) slabs below 128 filters pay only when one slab holds all filters.
    for (int ns = min_slabs; ns <= 16 && !P.resident; ++ns) {
      P.nslabs = ns;
      P.NT = slab_width(g.Co, ns, pair || fuse);
      P.NTh = pair ? P.NT / 2 : P.NT;
      if (P.NT < 128 && ns > 1) break;
      // (Lending four of the weight warps to the patch builders where a pixel has many channel
      // words was the better split while the drain loop was longer; since its trimming twelve
      // draining warps win on every layer measured: conv4 50.4 -> 48.1 us, conv5 39.4 -> 37.3.)
      P.wgt_warps = kWgtWarps;
      P.pat_group = kPatWarps;
      plan_stage(P);
      const int nst = (P.nsteps + P.mps - 1) / P.mps;
      if (nst <= kMaxBarStages && fits(nst, 2, 1)) {
        P.resident = 1;
        stages = nst; npb = 2;
        if (fits(stages, 3, 1)) npb = 3;
        if (npb == 3 && fits(stages, 4, 2)) npb = 4;     // a second raw buffer comes first
      }
    }
  }
  if (!P.resident) {
    P.nslabs = min_slabs;
    P.NT = slab_width(g.Co, P.nslabs, pair || fuse);
    P.NTh = pair ? P.NT / 2 : P.NT;
    P.wgt_warps = kWgtWarps;
    P.pat_group = kPatWarps;
    plan_stage(P);
    if (!fits(2, 1, 1)) return pl;
    // at least 2 stages and 1 patch; then patches up to 3, stages up to 6, one more patch
    stages = 2; npb = 1;
    while (stages < 4 && fits(stages + 1, npb, 1)) ++stages;
    while (npb < 3 && fits(stages, npb + 1, 1)) ++npb;
    while (stages < kMaxStages && fits(stages + 1, npb, 2)) ++stages;
    while (npb < kMaxPatchBufs && fits(stages, npb + 1, 2)) ++npb;
  }
  P.nraw = fits(stages, npb, 2) ? 2 : 1;
  P.nacc = std::max(1, std::min(kMaxAcc, kMaxAccCols / P.NT));
  // worker warps per quarter of the lanes in the resident schedule: the four epilogue warps
  // and the eight weight warps
  P.epi_split = std::min(kEpiSplitMax, P.NT / (fuse ? 32 : 16));
  if (fuse && (g.Co & 31) != 0) return pl;          // whole words of the next layer's input
  P.stages = stages; P.npb = npb;
  // small patches: every patch warp builds whole patches on its own, three at a time
  P.pat_sub = subgroups(npb);
  P.off_patch = P.off_ring + (uint32_t)stages * P.stage_bytes;
  P.off_raw = P.off_patch + (uint32_t)npb * P.patch_bytes;
  pl.smem = (size_t)P.off_raw + (size_t)(P.pat_sub * P.nraw) * P.raw_bytes;
  // block-scaled instruction descriptor: e2m1 x e2m1, ue8m0 scales, M = 128 (256 for a
  // pair), N = NT
  P.idesc = (1u << 7) | (1u << 10) | ((uint32_t)(P.NT >> 3) << 17) | (1u << 23) |
            ((uint32_t)((pair ? 2 * kTileM : kTileM) >> 4) << 24);
  const int crem = g.C - 32 * (g.Cw - 1);
  P.tail_mask = crem == 32 ? 0xFFFFFFFFu : ((1u << crem) - 1u);
  for (int j = 0; j < 32; ++j) P.swap_mask[j] = 0u;
  P.any_swap = 0;
  for (int j = 0; j < P.nsteps; ++j) {
    bool swap;
    P.adesc_lo[j] = kstep_desc(P, j, &swap);
    if (swap) { P.swap_mask[j >> 5] |= 1u << (j & 31); P.any_swap = 1; }
  }
  auto magic = [](uint32_t d, uint32_t *m, int *sh) {
    int l = 0;
    while ((1u << l) < d) ++l;
    *sh = l;
    *m = (uint32_t)((((unsigned long long)1 << (31 + l)) + d - 1) / d);
  };
  magic((uint32_t)P.Wq, &P.div_wq_m, &P.div_wq_s);
  magic((uint32_t)P.Hq, &P.div_hq_m, &P.div_hq_s);
  const uint32_t ngrp = (uint32_t)(P.Cw + 3) / 4u;
  magic((uint32_t)(s * s) * ngrp, &P.div_pg_m, &P.div_pg_s);
  magic(ngrp, &P.div_g_m, &P.div_g_s);
  pl.ok = true;
  return pl;
}

}  // namespace

namespace {

// The plan of a variant.  kTcAuto (measured on the AlexNet and ResNet-18 shapes): one CTA per
// SM unless only a pair, each CTA holding half of a slab, can keep the filters resident.
Plan plan_variant_uncached(const ConvGeom &g, TcVariant v, bool fuse) {
  switch (v) {
    case kTcSingle: return make_plan(g, 0, false, fuse);
    case kTcSingleStream: return make_plan(g, 1, false, fuse);
    case kTcPair: return make_plan(g, 0, true, fuse);
    case kTcPairStream: return make_plan(g, 1, true, fuse);
    default: break;
  }
  Plan single = make_plan(g, 0, false, fuse);
  if (single.ok && single.P.resident) return single;
  Plan pair = make_plan(g, 0, true, fuse);
  // neither resident: a pair pays when the slabs are wide (each CTA expands half the rows)
  if (pair.ok && (pair.P.resident || !single.ok || pair.P.NT > 128)) return pair;
  return single;
}

template <bool kRes, bool kPair, bool kFuse>
cudaError_t launch_variant(const Plan &pl, unsigned units, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kPair ? 2 * units : units);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kPair ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, binconv_tc_kernel<kRes, kPair, kFuse>, pl.P);
}

}  // namespace

// The last plans made, by (geometry, variant, fused): one call of the library plans its shape
// two or three times (support check, then launch), and a network repeats a few shapes; planning
// evaluates up to 800 descriptor words.  Plans hold no pointers until a launcher fills them in.
namespace {

struct PlanKey {
  int N, C, H, W, Co, kh, kw, stride, pad, variant, fuse;
  bool operator==(const PlanKey &o) const {
    return N == o.N && C == o.C && H == o.H && W == o.W && Co == o.Co && kh == o.kh && kw == o.kw &&
           stride == o.stride && pad == o.pad && variant == o.variant && fuse == o.fuse;
  }
};

Plan plan_variant(const ConvGeom &g, TcVariant v, bool fuse = false) {
  constexpr int kSlots = 16;
  static std::mutex mu;
  static PlanKey keys[kSlots];
  static Plan plans[kSlots];
  static bool used[kSlots] = {};
  static int next = 0;
  const PlanKey key{g.N, g.C, g.H, g.W, g.Co, g.kh, g.kw, g.stride, g.pad, (int)v, fuse ? 1 : 0};
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < kSlots; ++i)
    if (used[i] && keys[i] == key) return plans[i];
  const int slot = next;
  next = (next + 1) % kSlots;
  plans[slot] = plan_variant_uncached(g, v, fuse);
  keys[slot] = key;
  used[slot] = true;
  return plans[slot];
}

}  // namespace

bool umma_tc_supported(const ConvGeom &g, TcVariant v) { return plan_variant(g, v).ok; }

namespace {

cudaError_t launch_plan(Plan &pl, cudaStream_t st, bool fuse) {
  TcParams &P = pl.P;
  static bool attr_flags[64] = {};
  bool &attr_set = attr_done_for_current_device(attr_flags);
  if (!attr_set) {
    const void *kernels[8] = {(const void *)binconv_tc_kernel<false, false, false>,
                              (const void *)binconv_tc_kernel<true, false, false>,
                              (const void *)binconv_tc_kernel<false, true, false>,
                              (const void *)binconv_tc_kernel<true, true, false>,
                              (const void *)binconv_tc_kernel<false, false, true>,
                              (const void *)binconv_tc_kernel<true, false, true>,
                              (const void *)binconv_tc_kernel<false, true, true>,
                              (const void *)binconv_tc_kernel<true, true, true>};
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < 8 && e == cudaSuccess; ++i)
      e = cudaFuncSetAttribute(kernels[i], cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)kSmemMax);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  const long long total = (long long)P.ntiles * P.nslabs;
  const int sms = sm_count_of_current_device();
  // one CTA per SM, or one pair per two SMs
  const unsigned units = (unsigned)std::min<long long>(total, P.pair ? sms / 2 : sms);
  cudaError_t e_;
  if (fuse) {
    if (P.pair) e_ = P.resident ? launch_variant<true, true, true>(pl, units, st) : launch_variant<false, true, true>(pl, units, st);
    else e_ = P.resident ? launch_variant<true, false, true>(pl, units, st) : launch_variant<false, false, true>(pl, units, st);
  } else {
    if (P.pair) e_ = P.resident ? launch_variant<true, true, false>(pl, units, st) : launch_variant<false, true, false>(pl, units, st);
    else e_ = P.resident ? launch_variant<true, false, false>(pl, units, st) : launch_variant<false, false, false>(pl, units, st);
  }
  if (e_ != cudaSuccess) (void)cudaGetLastError();
  return e_;
}

}  // namespace

cudaError_t launch_binconv_tc(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                              const float *K, const float *residual, const ConvGeom &g,
                              const EpiOpts &epi, float *out, int32_t *acc_out, TcVariant variant,
                              cudaStream_t st) {
  Plan pl = plan_variant(g, variant);
  if (!pl.ok) return cudaErrorInvalidValue;
  TcParams &P = pl.P;
  P.xp = xp; P.wp = wp; P.alpha = alpha; P.K = K; P.residual = residual;
  P.out = out; P.acc_out = acc_out;
  P.relu = epi.relu; P.out_scale = epi.out_scale; P.acc_shift = epi.acc_shift; P.acc_accum = epi.acc_accum;
  P.nscale = nullptr; P.nshift = nullptr; P.xp_next = nullptr; P.A_part = nullptr; P.Cw_next = 0;
  return launch_plan(pl, st, false);
}

// Partial planes of |y| sums that the fused kernel writes for this shape: one per filter slab
// and, in the resident schedule, per warp that shares a quarter of the lanes.  0: not supported.
int tc_fused_parts(const ConvGeom &g, TcVariant variant) {
  const Plan pl = plan_variant(g, variant, true);
  if (!pl.ok) return 0;
  return pl.P.nslabs * (pl.P.resident ? pl.P.epi_split : 1);
}

cudaError_t launch_binconv_tc_fused(const uint32_t *xp, const uint32_t *wp, const float *alpha,
                                    const float *K, const float *residual, const ConvGeom &g,
                                    float *out, const float *next_scale, const float *next_shift,
                                    uint32_t *xp_next, float *A_part, TcVariant variant,
                                    cudaStream_t st) {
  Plan pl = plan_variant(g, variant, true);
  if (!pl.ok) return cudaErrorInvalidValue;
  TcParams &P = pl.P;
  P.xp = xp; P.wp = wp; P.alpha = alpha; P.K = K; P.residual = residual;
  P.out = out; P.acc_out = nullptr;
  P.relu = (g.flags & XNOR_FLAG_RELU) ? 1 : 0; P.out_scale = 1.0f; P.acc_shift = 0; P.acc_accum = 0;
  P.nscale = next_scale; P.nshift = next_shift; P.xp_next = xp_next; P.A_part = A_part;
  P.Cw_next = (g.Co + 31) / 32;
  return launch_plan(pl, st, true);
}


namespace {

// One warp waits, with a limit of about a millisecond, on a barrier that nothing signals: the
// wait must give up, raise the CTA's abort flag and record XNOR_ERR_TIMEOUT.
__global__ void wait_timeout_selftest_kernel() {
  __shared__ __align__(8) uint64_t bar;
  __shared__ volatile int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  (void)mbar_wait_slow(smem_u32(&bar), 0u, &abort_flag, &g_status_tc, 1ll << 21);
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(cudaStream_t st) {
  wait_timeout_selftest_kernel<<<1, 32, 0, st>>>();
  return cudaGetLastError();
}

cudaError_t read_status_tc(int *status) {
  cudaError_t e = cudaMemcpyFromSymbol(status, g_status_tc, sizeof(int));
  if (e == cudaSuccess && *status != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_status_tc, &zero, sizeof(int));
  }
#ifdef XNOR_BOUNDS_CHECK
  // checking build: a recorded violation wins over everything else (1000 + its site number)
  int site = 0;
  if (e == cudaSuccess) e = cudaMemcpyFromSymbol(&site, g_bounds_tc, sizeof(int));
  if (e == cudaSuccess && site != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbol(g_bounds_tc, &zero, sizeof(int));
    *status = 1000 + site;
  }
#endif
  return e;
}

}  // namespace xnor
