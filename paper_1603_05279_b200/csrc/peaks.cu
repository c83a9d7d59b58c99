// Measured peaks of the two pipes a binary convolution can run on (Section 4.1 counts the
// binary operations a processor performs per clock; these kernels measure that count here):
//   - tcgen05.mma kind::mxf4.block_scale on e2m1 operands resident in shared memory, the
//     instruction the tensor-core BinConv kernel issues, at the largest shape one CTA can issue
//     (128 x 256 x 64), so that the tensor pipe and not the issue rate bounds it;
//   - XOR + population count + add on the CUDA cores, the operation of the popcount kernel.
// Both report operations per SM clock, so the caller multiplies by the clock it observes.
#include <algorithm>

#include "common.cuh"
#include "umma_common.cuh"

namespace xnor {

namespace {

using namespace umma;

constexpr int kMaxBlocks = 256;
__device__ long long g_peak_cycles[kMaxBlocks];
__device__ int g_peak_status = 0;

constexpr int kMmaN = 256;
constexpr int kMmaIters = 16384;          // MMAs per block: ~2 M cycles, about a millisecond
constexpr int kMmaSmem = 64 * 1024;

__device__ __forceinline__ void mma_once(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc,
                                         uint32_t sf, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%4], [%4], p;\n\t}"
      ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(sf), "r"(accumulate) : "memory");
}

// One CTA per SM; operands are zeros in shared memory (the time of an MMA does not depend on
// the values), four A operands at different 16-byte offsets and four B operands, 128 x 256 x 64
// MMAs accumulating into tensor-memory columns 0-255.
__global__ void __launch_bounds__(128, 1) mma_rate_kernel() {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t slot;
  __shared__ volatile int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int i = tid; i < kMmaSmem / 16; i += 128) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
  if (tid == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = slot;
  {
    // unit block scales (ue8m0 1.0) in columns 480-511 of every lane
    const uint32_t taddr = tm + ((uint32_t)(warp * 32) << 16) + 480u;
    const uint32_t one = 0x7F7F7F7Fu;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};"
                   ::"r"(taddr + 8u * q), "r"(one) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    // e2m1 x e2m1, ue8m0 scales, M = 128, N = 256
    const uint32_t idesc = (1u << 7) | (1u << 10) | ((uint32_t)(kMmaN >> 3) << 17) | (1u << 23) |
                           ((uint32_t)(128 >> 4) << 24);
    const uint32_t a0 = smem_u32(smem), b0 = a0 + 16 * 1024;
    uint64_t ad[4], bd[4];
    for (int v = 0; v < 4; ++v) {
      ad[v] = make_desc(a0 + v * 16, 2560, 128);                     // A: 2 x (128 rows x 16 B)
      bd[v] = make_desc(b0 + v * 8192, (uint32_t)kMmaN * 16, 128);    // B: 2 x (256 rows x 16 B)
    }
    const long long t0 = clock64();
    for (int i = 0; i < kMmaIters / 4; ++i) {
#pragma unroll
      for (int v = 0; v < 4; ++v) mma_once(tm, ad[v], bd[v], idesc, tm + 480u, 1u);
    }
    umma_commit(smem_u32(&bar));
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, &g_peak_status);
    const long long t1 = clock64();
    if (blockIdx.x < kMaxBlocks) g_peak_cycles[blockIdx.x] = ok ? t1 - t0 : -1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(512u) : "memory");
}

constexpr int kPopcThreads = 1024;
constexpr int kPopcIters = 2048;
constexpr int kPopcChains = 8;

// Every thread runs 8 independent chains of acc += popc(x ^ y), y changing every step.
__global__ void __launch_bounds__(kPopcThreads, 1) popc_rate_kernel(uint32_t seed, uint32_t *sink) {
  uint32_t x[kPopcChains], acc[kPopcChains];
#pragma unroll
  for (int c = 0; c < kPopcChains; ++c) { x[c] = seed * (threadIdx.x + 1u) + 0x9E3779B9u * c; acc[c] = 0u; }
  uint32_t y = seed ^ threadIdx.x;
  __syncthreads();
  const long long t0 = clock64();
#pragma unroll 4
  for (int i = 0; i < kPopcIters; ++i) {
#pragma unroll
    for (int c = 0; c < kPopcChains; ++c) acc[c] += __popc(x[c] ^ y);
    y = y * 1664525u + 1013904223u;
  }
  const long long t1 = clock64();
  uint32_t s = 0;
#pragma unroll
  for (int c = 0; c < kPopcChains; ++c) s += acc[c];
  if (s == 0x12345678u) *sink = s;                    // keeps the chains alive
  __syncthreads();
  if (threadIdx.x == 0 && blockIdx.x < kMaxBlocks) g_peak_cycles[blockIdx.x] = t1 - t0;
}

__device__ uint32_t g_popc_sink;

// median of the positive per-block cycle counts
cudaError_t median_cycles(int blocks, double *cycles) {
  long long h[kMaxBlocks];
  cudaError_t e = cudaMemcpyFromSymbol(h, g_peak_cycles, sizeof(long long) * blocks);
  if (e != cudaSuccess) return e;
  std::sort(h, h + blocks);
  if (h[0] <= 0) return cudaErrorUnknown;              // a wait gave up
  *cycles = (double)h[blocks / 2];
  return cudaSuccess;
}

}  // namespace

cudaError_t measure_pipe_peaks(double *mma_mac_per_clk_per_sm, double *popc_per_clk_per_sm,
                               cudaStream_t st) {
  const int blocks = std::min(sm_count_of_current_device(), kMaxBlocks);
  static bool attr_flags[64] = {};
  bool &attr_set = attr_done_for_current_device(attr_flags);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMmaSmem);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e; }
    attr_set = true;
  }
  cudaError_t e;
  double cyc = 0.0;
  // twice: the first launch warms the clocks and the instruction cache
  for (int rep = 0; rep < 2; ++rep) {
    mma_rate_kernel<<<blocks, 128, kMmaSmem, st>>>();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return e;
  }
  if ((e = median_cycles(blocks, &cyc)) != cudaSuccess) return e;
  *mma_mac_per_clk_per_sm = 128.0 * kMmaN * 64.0 * kMmaIters / cyc;
  uint32_t *sink = nullptr;
  if ((e = cudaGetSymbolAddress((void **)&sink, g_popc_sink)) != cudaSuccess) return e;
  for (int rep = 0; rep < 2; ++rep) {
    popc_rate_kernel<<<blocks, kPopcThreads, 0, st>>>(12345u + rep, sink);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return e;
  }
  if ((e = median_cycles(blocks, &cyc)) != cudaSuccess) return e;
  *popc_per_clk_per_sm = (double)kPopcThreads * kPopcChains * kPopcIters / cyc;
  return cudaSuccess;
}

}  // namespace xnor
