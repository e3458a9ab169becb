// Microbenchmark of the tcgen05.mma forms the tile kernels use: cycles per group of 8 MMAs (M = 128, K = 8 x 16, bf16,
// fp32 accumulators in TMEM) for each operand source (A from shared memory or TMEM, B K-major or MN-major) and N = 64,
// 128, 256, alone and with three warps reading shared memory beside the issuing thread.  One CTA per SM, every wait
// bounded.  Not part of the library.  Build and run:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o probe_mma_rate paper_2609_33133_b200/csrc/probe_mma_rate.cu && ./probe_mma_rate
#include <cstdio>
#include <type_traits>
#include <cuda_runtime.h>
#include "ptx.cuh"
using namespace augtree;

__global__ void __launch_bounds__(128, 1) probe(long long *out, int *status, int rounds, int bg_gap) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t base = smem_u32(smem);
  const uint32_t sA = base, sB = base + 32768, sB2 = base + 65536, bar = base + 98304;
  volatile uint32_t *slot = reinterpret_cast<volatile uint32_t *>(smem + 98304 + 16);
  volatile int *flag = reinterpret_cast<volatile int *>(smem + 98304 + 24);
  for (int i = threadIdx.x; i < 98304 / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(smem)[i] = 0x3c003c00u;
  if (threadIdx.x == 0) { mbar_init(bar, 1); *flag = 0; *reinterpret_cast<volatile int *>(smem + 98304 + 32) = 0; fence_barrier_init(); }
  const int warp = threadIdx.x >> 5;
  if (warp == 0) { tmem_alloc(smem_u32((const void *)slot), 512); tmem_relinquish(); }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *slot;
  AbortCtx ab{flag, status, 1ll << 28};
  if (threadIdx.x == 0) {
    const uint32_t a_k = sdesc_lo(sA, 16), b_k = sdesc_lo(sB, 16), b_mn = sdesc_lo(sB, 16384), a_mn = sdesc_lo(sA, 16384);
    uint32_t phase = 0;
    auto run = [&](auto tag) {
      constexpr int variant = decltype(tag)::value;
      const long long t0 = clock64();
      for (int r = 0; r < rounds; ++r) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t acc = (r > 0 || k > 0);
          if constexpr (variant == 0) mma_ss2(tmem + 256, a_k + kstep_kmajor(k), b_k + kstep_kmajor(k), make_idesc(128, 128, 0, 0), acc);
          if constexpr (variant == 1) mma_ts2(tmem + 256, tmem + 8 * k, b_k + kstep_kmajor(k), make_idesc(128, 128, 0, 0), acc);
          if constexpr (variant == 2) mma_ts2(tmem + 256, tmem + 8 * k, b_mn + kstep_mnmajor(k), make_idesc(128, 128, 0, 1), acc);
          if constexpr (variant == 3) mma_ss2(tmem + 256, a_k + kstep_kmajor(k), b_k + kstep_kmajor(k), make_idesc(128, 64, 0, 0), acc);
          if constexpr (variant == 4) mma_ss2(tmem + 256, a_mn + kstep_mnmajor(k), b_mn + kstep_mnmajor(k), make_idesc(128, 128, 1, 1), acc);
          if constexpr (variant == 5) mma_ss2(tmem + 256, a_k + kstep_kmajor(k), b_k + kstep_kmajor(k), make_idesc(128, 256, 0, 0), acc);
          if constexpr (variant == 6) mma_ts2(tmem + 256, tmem + 8 * k, b_k + kstep_kmajor(k), make_idesc(128, 64, 0, 0), acc);
          if constexpr (variant == 7) mma_ss2(tmem + 256, a_k + kstep_kmajor(k), b_mn + kstep_mnmajor(k), make_idesc(128, 128, 0, 1), acc);
        }
      }
      tc_commit(bar);
      const bool ok = mbar_wait(bar, phase & 1, ab, 99);
      ++phase;
      const long long t1 = clock64();
      if (blockIdx.x == 0) out[variant] = t1 - t0;
      return ok;
    };
    bool ok = run(std::integral_constant<int, 0>{});
    ok = ok && run(std::integral_constant<int, 1>{});
    ok = ok && run(std::integral_constant<int, 2>{});
    ok = ok && run(std::integral_constant<int, 3>{});
    ok = ok && run(std::integral_constant<int, 4>{});
    ok = ok && run(std::integral_constant<int, 5>{});
    ok = ok && run(std::integral_constant<int, 6>{});
    ok = ok && run(std::integral_constant<int, 7>{});
  }
  else if (bg_gap >= 0 && warp > 0) {
    // background shared-memory traffic: every lane of warps 1-3 reads 16 bytes (512 contiguous bytes per warp
    // instruction = 4 wavefronts), then idles bg_gap clocks
    volatile int *done = reinterpret_cast<volatile int *>(smem + 98304 + 32);
    uint32_t sink = 0;
    const uint4 *src = reinterpret_cast<const uint4 *>(smem + 65536) + (threadIdx.x & 31);
    long long guard = 0;
    while (!*done && guard < (1ll << 26)) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        uint32_t a, b, c, d;
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(smem_u32(src + 32 * i)));
        sink += a + d;
      }
      if (bg_gap > 0) { const long long t = clock64(); while (clock64() - t < bg_gap) {} }
      guard += 1;
    }
    if (sink == 0x12345678u) out[15] = sink;
  }
  if (threadIdx.x == 0) *reinterpret_cast<volatile int *>(smem + 98304 + 32) = 1;
  __syncthreads();
  if (warp == 0) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

int main() {
  long long *out; int *status;
  cudaMalloc(&out, 16 * sizeof(long long)); cudaMalloc(&status, 16 * sizeof(int));
  cudaMemset(out, 0, 8 * sizeof(long long)); cudaMemset(status, 0, 16 * sizeof(int));
  cudaFuncSetAttribute(probe, cudaFuncAttributeMaxDynamicSharedMemorySize, 99328);
  const int rounds = 2000;
  for (int bg : {-1, 0, 64, 256, 1024}) {
    const int grid = 148;
    probe<<<grid, 128, 99328>>>(out, status, rounds, bg);
    cudaError_t e = cudaDeviceSynchronize();
    long long h[8]; int st[2];
    cudaMemcpy(h, out, sizeof(h), cudaMemcpyDeviceToHost); cudaMemcpy(st, status, sizeof(st), cudaMemcpyDeviceToHost);
    printf("background gap %d: %s status %d %d\n", bg, cudaGetErrorString(e), st[0], st[1]);
    const char *names[8] = {"SS K/K N=128", "TS B K-major N=128", "TS B MN-major N=128", "SS N=64", "SS MN/MN N=128", "SS N=256", "TS N=64", "SS A K-major B MN-major"};
    for (int v = 0; v < 8; ++v) printf("  %-26s %8.1f cycles per 8-MMA group\n", names[v], (double)h[v] / rounds);
  }
  return 0;
}
