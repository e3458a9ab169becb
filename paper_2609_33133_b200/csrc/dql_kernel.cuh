// Backward, query side (dQ) from handed-over dS: one persistent CTA per replay lane walks its list of
// (query tile, head) items, the same items and the same summation order as dq_kernel.  The key-side kernel
// has already stored dS^T of every (KV tile, query tile, head) pair as a bf16 tile, so what is left of
//   dQ = sum over the KV tiles T the queries see of  dS(T) K(T)                     (Eq. 1's backward)
// is one GEMM per pair: A = dS(T) read MN-major from the stored [keys][queries] tile, B = K(T) MN-major.
// No exponentials, no statistics, no Q, dO or V: the kernel streams 32 KB of dS per 128 x 128 x D MMA
// group and is bound by HBM (dS is written and read once; K tiles come from L2).
//
// Warp roles (192 threads): warps 0-3 epilogue (thread = query row), warp 4 lane 0 TMA loads, warp 5 MMA
// issue.  TMEM: two dQ accumulators (columns 0 and 128), so that an item's epilogue runs under the next item.
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace augtree {

struct DqlParams {
  const int32_t *items;     // lane order, 12 ints (query-side items)
  const int32_t *lane_ptr;  // [gridDim.x + 1]
  const int4 *pair_tab;     // per query tile {first slot / h_q, KV tiles seen, prompt KV tiles among them, 0}
  __nv_bfloat16 *dq;        // [query tokens, h_q, D]
  float *dq_f32;            // partial-state variant: dQ is written here in fp32
  int h_q;
  int d;                    // head dimension of the tensors (<= D)
  int no_own;               // partial-state variant: the causal range of the query's own sequence is left out
  int *status;
  long long wait_budget;
  int kind;
};

constexpr int kDqlThreads = 192;

template <int D>
struct DqlSmem {
  static constexpr int kStages = 3;
  static constexpr int kDsBytes = 128 * 128 * 2, kKBytes = 128 * D * 2;
  static constexpr int kStageBytes = kDsBytes + kKBytes;
  static constexpr int kOffBar = kStages * kStageBytes;
  static constexpr int kBytes = kOffBar + 128;
};

enum : int { WAIT_DQL_FULL = 60, WAIT_DQL_EMPTY = 61, WAIT_DQL_ACC_FULL = 62, WAIT_DQL_ACC_EMPTY = 63 };

template <int D>
__global__ void __launch_bounds__(kDqlThreads, 1)
dql_kernel(const __grid_constant__ CUtensorMap tm_ds, const __grid_constant__ CUtensorMap tm_ka,
           const __grid_constant__ CUtensorMap tm_kb, const DqlParams p) {
  using SM = DqlSmem<D>;
  constexpr int NBOX = D / 64;
  constexpr int NST = SM::kStages;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {
    if (threadIdx.x == 0 && atomicCAS(p.status, 0, -6) == 0) p.status[1] = 3;
    return;
  }
  const uint32_t bars = base + SM::kOffBar;
  const uint32_t bar_full = bars, bar_empty = bars + 32;          // [NST <= 4]
  const uint32_t bar_acc_full = bars + 64, bar_acc_empty = bars + 80;  // [2]
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_raw + SM::kOffBar + 96);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + SM::kOffBar + 104);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < NST; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(bar_acc_full + 8 * s, 1); mbar_init(bar_acc_empty + 8 * s, 4); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 5) { tmem_alloc(smem_u32((const void *)tmem_slot), 256); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const AbortCtx ab{abort_flag, p.status, p.wait_budget};
  const int it_begin = p.lane_ptr[blockIdx.x], it_end = p.lane_ptr[blockIdx.x + 1];

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_ds); tma_prefetch_desc(&tm_ka); tma_prefetch_desc(&tm_kb);
      const uint64_t pol_first = policy_evict_first();
      uint32_t T = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const int32_t *I = p.items + (size_t)it * 12;
        const int head = I[3], a_tok0 = I[4], a_len = I[5], b_tok0 = I[6], tile = I[8], kvh = I[11];
        const int b_len = p.no_own ? 0 : I[7];
        const int nA = (a_len + 127) >> 7, n = nA + ((b_len + 127) >> 7);
        const int4 pt = __ldg(p.pair_tab + tile);
        const long long slot0 = (long long)pt.x * p.h_q + (long long)head * pt.y;
        for (int j = 0; j < n && ok; ++j, ++T) {
          const uint32_t st = T % NST;
          ok = mbar_wait(bar_empty + 8 * st, ((T / NST) & 1) ^ 1, ab, WAIT_DQL_EMPTY);
          if (!ok) break;
          const uint32_t sDs = base + st * SM::kStageBytes, sK = sDs + SM::kDsBytes;
          mbar_expect_tx(bar_full + 8 * st, SM::kStageBytes);
          // (the stored tile's slot: the prompt KV tiles come first, then the sequence's own)
          tma_load_3d_hint(sDs, &tm_ds, bar_full + 8 * st, 0, 0, (int)(slot0 + j), pol_first);   // read once
          tma_load_3d_hint(sDs + 16384, &tm_ds, bar_full + 8 * st, 64, 0, (int)(slot0 + j), pol_first);
          const bool in_a = j < nA;
          const int row = in_a ? a_tok0 + j * 128 : b_tok0 + (j - nA) * 128;
          for (int b = 0; b < NBOX; ++b) tma_load_3d(sK + b * 16384, in_a ? &tm_ka : &tm_kb, bar_full + 8 * st, b * 64, kvh, row);
        }
      }
    }
  } else if (warp == 5) {
    // -------------------------------------------------------------- MMA issuer
    constexpr uint32_t IDESC = make_idesc(128, D, 1, 1);  // A = dS MN-major (queries contiguous), B = K MN-major
    const bool elected = elect_one();
    const int it_b = __shfl_sync(0xffffffffu, it_begin, 0), it_e = __shfl_sync(0xffffffffu, it_end, 0);
    uint32_t ic = 0, T = 0;
    bool ok = true;
    for (int it = it_b; it < it_e && ok; ++it, ++ic) {
      const int32_t *I = p.items + (size_t)it * 12;
      const int n = __shfl_sync(0xffffffffu, ((I[5] + 127) >> 7) + (p.no_own ? 0 : ((I[7] + 127) >> 7)), 0);
      const uint32_t buf = ic & 1;
      if (ic >= 2) {  // the accumulator's previous item must have left TMEM
        ok = mbar_wait(bar_acc_empty + 8 * buf, ((ic >> 1) - 1) & 1, ab, WAIT_DQL_ACC_EMPTY);
        if (!ok) break;
        tc_fence_after();
      }
      const uint32_t tDQ = tmem + buf * 128;
      for (int j = 0; j < n && ok; ++j, ++T) {
        const uint32_t st = T % NST;
        ok = mbar_wait(bar_full + 8 * st, (T / NST) & 1, ab, WAIT_DQL_FULL);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sDs = base + st * SM::kStageBytes;
        const uint32_t a_lo = sdesc_lo(sDs, 16384), b_lo = sdesc_lo(sDs + SM::kDsBytes, 16384);
        if (elected) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ss2(tDQ, a_lo + kstep_mnmajor(k), b_lo + kstep_mnmajor(k), IDESC, (uint32_t)(j > 0 || k > 0));
          tc_commit(bar_empty + 8 * st);
        }
      }
      if (!ok) break;
      if (elected) tc_commit(bar_acc_full + 8 * buf);
    }
  } else {
    // ------------------------------------------------------------ epilogue warps 0-3
    const int r = warp * 32 + lane;  // TMEM lane = query row of the tile
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    uint32_t ic = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
      const int32_t *I = p.items + (size_t)it * 12;
      const int q_tok0 = I[0], q_rows = I[2], head = I[3];
      const uint32_t buf = ic & 1;
      ok = mbar_wait(bar_acc_full + 8 * buf, (ic >> 1) & 1, ab, WAIT_DQL_ACC_FULL);
      if (!ok) break;
      tc_fence_after();
      const long long row_off = (((long long)q_tok0 + r) * p.h_q + head) * p.d;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(tmem + buf * 128 + lane_off + c * 32, v);
        tc_wait_ld();
        if (r < q_rows && p.dq_f32) {
          float4 *dst = reinterpret_cast<float4 *>(p.dq_f32 + row_off + c * 32);
#pragma unroll
          for (int e = 0; e < 8; ++e)
            if (c * 32 + 4 * e < p.d) dst[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]), __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
        } else if (r < q_rows) {
          uint4 *dst = reinterpret_cast<uint4 *>(p.dq + row_off + c * 32);
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (c * 32 + 8 * e < p.d) dst[e] = make_uint4(pack_bf16(__uint_as_float(v[8 * e]), __uint_as_float(v[8 * e + 1])),
                                pack_bf16(__uint_as_float(v[8 * e + 2]), __uint_as_float(v[8 * e + 3])),
                                pack_bf16(__uint_as_float(v[8 * e + 4]), __uint_as_float(v[8 * e + 5])),
                                pack_bf16(__uint_as_float(v[8 * e + 6]), __uint_as_float(v[8 * e + 7])));
        }
      }
      tc_fence_before();
      warp_arrive(bar_acc_empty + 8 * buf);
      if (warp == 0 && lane == 0) atomicAdd(p.status + 2 + p.kind, 1);  // item finished (work accounting)
    }
  }

  __syncwarp();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) {}
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem, 256); }
}

}  // namespace augtree
