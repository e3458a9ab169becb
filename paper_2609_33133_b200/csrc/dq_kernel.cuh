// Backward, query side (dQ), query-stationary: one persistent CTA per replay lane
// walks its list of (query tile, head) items.  An item keeps its Q and dO tile in
// TMEM (as bf16 A operands) and its dQ accumulator in TMEM, and streams past them
// the KV tiles the queries can see: the unmasked shared prompt range, then the
// causal range of the query's own sequence (Eq. 1).  dQ therefore needs no
// atomics: every (query tile, head) has one owner and a fixed summation order.
//
// Per KV tile T:
//   S   = Q K^T              (A = Q from TMEM, B = K K-major)
//   P   = exp2(S * scale*log2e - lse2[q])            (element-wise warps, registers only)
//   dP  = dO V^T             (A = dO from TMEM, B = V K-major)
//   dS  = P * (scale*dP - scale*delta[q])            (bf16, written over dP in TMEM)
//   dQ += dS K               (A = dS from TMEM, B = the same K tile read MN-major)
//
// Warp roles (320 threads): warps 0-7 element-wise (warp w: TMEM lanes = query rows
// 32*(w%4).., key columns 64*(w/4)..), warp 8 lane 0 TMA loads, warp 9 lane 0 MMA issue.
// TMEM columns: Q at 0, dO at D/2 (bf16 pairs), S at 128, dP/dS at 256, dQ at 384.
// MMA issue order in steady state: S(T+1), dQ(T), dP(T+1).
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace augtree {

struct DqParams {
  const int32_t *items;     // lane order, 12 ints: q_tok0, q_pos0, q_rows, head, a_tok0, a_len, b_tok0, b_len,
                            //                      stats tile index, 1, weight, kv head
  const int32_t *lane_ptr;  // [gridDim.x + 1]
  const float *stats;       // [h_q][n_tiles][2][128]: -lse*log2e (-inf past the end), -scale*rowsum(dO*O)
  __nv_bfloat16 *dq;        // [query tokens, h_q, D]
  long long n_tiles;
  int h_q;
  int d;                    // head dimension of the tensors (<= D)
  float scale, scale_log2;
  int *status;
  long long wait_budget;    // clocks a wait may take before the kernel gives up
  int kind;                 // schedule index: status[2 + kind] counts finished items
  int no_own;               // partial-state variant: the causal range of the query's own sequence is left out
  float *dq_f32;            // partial-state variant: dQ is written here in fp32 (summed over KV owners afterwards)
};

constexpr int kDqThreads = 320;
#ifndef AUGTREE_DQ_FMA_MASK
#define AUGTREE_DQ_FMA_MASK 0x8888u
#endif
constexpr uint32_t kDqFmaMask = AUGTREE_DQ_FMA_MASK;  // pairs (period 16) whose exp2 runs on the FMA pipe

template <int D>
struct DqSmem {
  static constexpr int kNK = 3, kNV = 2;  // K and V rings
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kOffQ = 0, kOffDo = kTileBytes;
  static constexpr int kOffK = 2 * kTileBytes;              // [kNK]
  static constexpr int kOffV = kOffK + kNK * kTileBytes;    // [kNV]
  static constexpr int kOffStats = kOffV + kNV * kTileBytes;  // [2][128] floats
  static constexpr int kOffBar = kOffStats + 1024;
  static constexpr int kBytes = kOffBar + 256;
};

enum : int { WAIT_DQ_QDO = 50, WAIT_DQ_QT = 51, WAIT_DQ_K = 52, WAIT_DQ_V = 53, WAIT_DQ_S = 54, WAIT_DQ_SREAD = 55,
             WAIT_DQ_DP = 56, WAIT_DQ_DS = 57, WAIT_DQ_FULL = 58, WAIT_DQ_EMPTY = 59 };

template <int D>
__global__ void __launch_bounds__(kDqThreads, 1)
dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
          const __grid_constant__ CUtensorMap tm_ka, const __grid_constant__ CUtensorMap tm_va,
          const __grid_constant__ CUtensorMap tm_kb, const __grid_constant__ CUtensorMap tm_vb, const DqParams p) {
  using SM = DqSmem<D>;
  constexpr int TILE = SM::kTileBytes;
  constexpr int NBOX = D / 64;
  constexpr int NK = SM::kNK, NV = SM::kNV;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {
    if (threadIdx.x == 0 && atomicCAS(p.status, 0, -6) == 0) p.status[1] = 2;
    return;
  }
  const uint32_t sQ = base + SM::kOffQ, sDo = base + SM::kOffDo, sK0 = base + SM::kOffK, sV0 = base + SM::kOffV;
  const uint32_t sStats = base + SM::kOffStats;
  const uint32_t bars = base + SM::kOffBar;
  const uint32_t bar_qdo_full = bars, bar_qdo_empty = bars + 8, bar_qt_ready = bars + 16;
  const uint32_t bar_k_full = bars + 24, bar_k_empty = bars + 56;  // [NK <= 4]
  const uint32_t bar_v_full = bars + 88, bar_v_empty = bars + 120; // [NV <= 4]
  const uint32_t bar_s_full = bars + 152, bar_s_read = bars + 160, bar_dp_full = bars + 168, bar_ds_ready = bars + 176;
  const uint32_t bar_dq_full = bars + 184, bar_dq_empty = bars + 192;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_raw + SM::kOffBar + 200);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + SM::kOffBar + 208);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar_qdo_full, 1); mbar_init(bar_qdo_empty, 8); mbar_init(bar_qt_ready, 8);
    for (int s = 0; s < NK; ++s) { mbar_init(bar_k_full + 8 * s, 1); mbar_init(bar_k_empty + 8 * s, 1); }
    for (int s = 0; s < NV; ++s) { mbar_init(bar_v_full + 8 * s, 1); mbar_init(bar_v_empty + 8 * s, 1); }
    mbar_init(bar_s_full, 1); mbar_init(bar_s_read, 8); mbar_init(bar_dp_full, 1); mbar_init(bar_ds_ready, 8);
    mbar_init(bar_dq_full, 1); mbar_init(bar_dq_empty, 8);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 9) { tmem_alloc(smem_u32((const void *)tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tQ = tmem, tDO = tmem + D / 2, tS = tmem + 128, tDP = tmem + 256, tDQ = tmem + 384;
  const AbortCtx ab{abort_flag, p.status, p.wait_budget};
  const int it_begin = p.lane_ptr[blockIdx.x], it_end = p.lane_ptr[blockIdx.x + 1];

  if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_do); tma_prefetch_desc(&tm_ka);
      tma_prefetch_desc(&tm_va); tma_prefetch_desc(&tm_kb); tma_prefetch_desc(&tm_vb);
      uint32_t ic = 0, T = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
        const int32_t *I = p.items + (size_t)it * 12;
        const int q_tok0 = I[0], head = I[3], a_tok0 = I[4], a_len = I[5], b_tok0 = I[6], tile = I[8], kvh = I[11];
        const int b_len = p.no_own ? 0 : I[7];
        const int nA = (a_len + 127) >> 7, n = nA + ((b_len + 127) >> 7);
        ok = mbar_wait(bar_qdo_empty, (ic & 1) ^ 1, ab, WAIT_DQ_QDO);
        if (!ok) break;
        mbar_expect_tx(bar_qdo_full, 2 * TILE + 1024);
        for (int b = 0; b < NBOX; ++b) {
          tma_load_3d(sQ + b * 16384, &tm_q, bar_qdo_full, b * 64, head, q_tok0);
          tma_load_3d(sDo + b * 16384, &tm_do, bar_qdo_full, b * 64, head, q_tok0);
        }
        bulk_load_1d(sStats, p.stats + ((long long)head * p.n_tiles + tile) * 256, 1024, bar_qdo_full);
        for (int j = 0; j < n && ok; ++j, ++T) {
          const bool in_a = j < nA;
          const int row = in_a ? a_tok0 + j * 128 : b_tok0 + (j - nA) * 128;
          const uint32_t ks = T % NK, vs = T % NV;
          ok = mbar_wait(bar_k_empty + 8 * ks, ((T / NK) & 1) ^ 1, ab, WAIT_DQ_K);
          if (!ok) break;
          mbar_expect_tx(bar_k_full + 8 * ks, TILE);
          for (int b = 0; b < NBOX; ++b) tma_load_3d(sK0 + ks * TILE + b * 16384, in_a ? &tm_ka : &tm_kb, bar_k_full + 8 * ks, b * 64, kvh, row);
          ok = mbar_wait(bar_v_empty + 8 * vs, ((T / NV) & 1) ^ 1, ab, WAIT_DQ_V);
          if (!ok) break;
          mbar_expect_tx(bar_v_full + 8 * vs, TILE);
          for (int b = 0; b < NBOX; ++b) tma_load_3d(sV0 + vs * TILE + b * 16384, in_a ? &tm_va : &tm_vb, bar_v_full + 8 * vs, b * 64, kvh, row);
        }
      }
    }
  } else if (warp == 9) {
    // -------------------------------------------------------------- MMA issuer
    // The whole warp runs the loops in lockstep and one elected lane issues (warp-uniform descriptor
    // arithmetic keeps the instruction count per MMA small next to two busy element-wise warps on the
    // same scheduler); each group looks at the next group's barrier before its own last two MMAs.
    {
      constexpr uint32_t IDESC_S = make_idesc(128, 128, 0, 0);  // S, dP: A from TMEM, B K-major
      constexpr uint32_t IDESC_DQ = make_idesc(128, D, 0, 1);   // dQ: A = dS from TMEM, B = K MN-major
      constexpr int NKS = D / 16;
      const bool elected = elect_one();
      const int it_b = __shfl_sync(0xffffffffu, it_begin, 0), it_e = __shfl_sync(0xffffffffu, it_end, 0);
      uint32_t ic = 0, T = 0;
      bool ok = true;
      auto need = [&](bool have, uint32_t bar, uint32_t par, int site) -> bool {
        if (!have && !mbar_wait(bar, par, ab, site)) return false;
        tc_fence_after();
        return true;
      };
      // S(Tn) = Q K^T; `look` runs before the last two MMAs
      auto issue_s = [&](uint32_t Tn, bool have, auto look) -> bool {
        const uint32_t ks = Tn % NK;
        if (!need(have, bar_k_full + 8 * ks, (Tn / NK) & 1, WAIT_DQ_K)) return false;
        const uint32_t k_lo = sdesc_lo(sK0 + ks * TILE, 16);
        mma_group<NKS>(elected, [&](int k) { mma_ts2(tS, tQ + k * 8, k_lo + kstep_kmajor(k), IDESC_S, k > 0); }, look);
        if (elected) tc_commit(bar_s_full);
        return true;
      };
      // dP(Tn) = dO V^T
      auto issue_dp = [&](uint32_t Tn, bool have, auto look) -> bool {
        const uint32_t vs = Tn % NV;
        if (!need(have, bar_v_full + 8 * vs, (Tn / NV) & 1, WAIT_DQ_V)) return false;
        const uint32_t v_lo = sdesc_lo(sV0 + vs * TILE, 16);
        mma_group<NKS>(elected, [&](int k) { mma_ts2(tDP, tDO + k * 8, v_lo + kstep_kmajor(k), IDESC_S, k > 0); }, look);
        if (elected) { tc_commit(bar_dp_full); tc_commit(bar_v_empty + 8 * vs); }
        return true;
      };
      for (int it = it_b; it < it_e && ok; ++it, ++ic) {
        const int32_t *I = p.items + (size_t)it * 12;
        const int n = __shfl_sync(0xffffffffu, ((I[5] + 127) >> 7) + (p.no_own ? 0 : ((I[7] + 127) >> 7)), 0);
        ok = mbar_wait(bar_qt_ready, ic & 1, ab, WAIT_DQ_QT);
        if (!ok) break;
        bool have_sread = false, have_ds = false, have_v = false, have_k = false;
        ok = issue_s(T, false, [&]() { have_v = mbar_test(bar_v_full + 8 * (T % NV), (T / NV) & 1); }) &&
             issue_dp(T, have_v, [&]() { have_sread = n > 1 && mbar_test(bar_s_read, T & 1); });
        for (int i = 0; i < n && ok; ++i, ++T) {
          const bool more = i + 1 < n;
          have_ds = false;
          if (more) {  // S(T+1): the warps must have read S(T) out of TMEM
            ok = need(have_sread, bar_s_read, T & 1, WAIT_DQ_SREAD);
            if (!ok) break;
            have_k = mbar_test(bar_k_full + 8 * ((T + 1) % NK), ((T + 1) / NK) & 1);
            ok = issue_s(T + 1, have_k, [&]() { have_ds = mbar_test(bar_ds_ready, T & 1); });
            if (!ok) break;
          }
          // dQ += dS(T) K(T)
          ok = need(have_ds, bar_ds_ready, T & 1, WAIT_DQ_DS);
          if (!ok) break;
          if (i == 0 && ic > 0) {  // the previous item's dQ must have left TMEM
            ok = need(false, bar_dq_empty, (ic - 1) & 1, WAIT_DQ_EMPTY);
            if (!ok) break;
          }
          const uint32_t ks = T % NK;
          const uint32_t km_lo = sdesc_lo(sK0 + ks * TILE, 16384);
          const uint32_t acc0 = i > 0 ? 1u : 0u;
          have_v = false;
          // (key columns 16k..16k+15: dS sits at dP columns 8k (k<4) or 64+8(k-4))
          mma_group<8>(elected,
                       [&](int k) {
                         mma_ts2(tDQ, tDP + (k < 4 ? k * 8 : 64 + (k - 4) * 8), km_lo + kstep_mnmajor(k), IDESC_DQ, acc0 | (uint32_t)(k > 0));
                       },
                       [&]() { have_v = more && mbar_test(bar_v_full + 8 * ((T + 1) % NV), ((T + 1) / NV) & 1); });
          if (elected) tc_commit(bar_k_empty + 8 * ks);
          have_sread = false;
          if (more)  // dP(T+1) overwrites dS(T): the tensor pipe runs in order
            ok = issue_dp(T + 1, have_v, [&]() { have_sread = i + 2 < n && mbar_test(bar_s_read, (T + 1) & 1); });
        }
        if (!ok) break;
        if (elected) tc_commit(bar_dq_full);
      }
    }
  } else {
    // ------------------------------------------------------- element-wise warps 0-7
    const int lg = warp & 3, ch = warp >> 2;
    const int r = lg * 32 + lane;  // TMEM lane = query row of the tile
    const uint32_t lane_off = (uint32_t)(lg * 32) << 16;
    uint32_t ic = 0, T = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
      const int32_t *I = p.items + (size_t)it * 12;
      const int q_tok0 = I[0], q_pos0 = I[1], q_rows = I[2], head = I[3], a_len = I[5];
      const int b_len = p.no_own ? 0 : I[7];
      const int nA = (a_len + 127) >> 7, n = nA + ((b_len + 127) >> 7);
      // ---- Q and dO rows into TMEM as bf16 A operands; this thread: row r, columns (D/2)*ch .. of d
      ok = mbar_wait(bar_qdo_full, ic & 1, ab, WAIT_DQ_QDO);
      if (!ok) break;
      const float nlse2 = reinterpret_cast<const float *>(smem_raw + SM::kOffStats)[r];        // -lse * log2(e)
      const float ndlt = reinterpret_cast<const float *>(smem_raw + SM::kOffStats)[128 + r];   // -scale * delta
      {
        constexpr int NCH = D / 16;  // 16-byte chunks per thread (8 for D=128: one whole box; 4 for D=64: half a box)
        const int box = (D == 128) ? ch : 0, c0 = (D == 128) ? 0 : ch * 4;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
          const uint8_t *row = smem_raw + (which ? SM::kOffDo : SM::kOffQ) + box * 16384 + r * 128;
          uint32_t w[NCH * 4];
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            const uint4 x = *reinterpret_cast<const uint4 *>(row + (((c0 + c) ^ (r & 7)) << 4));
            w[4 * c] = x.x; w[4 * c + 1] = x.y; w[4 * c + 2] = x.z; w[4 * c + 3] = x.w;
          }
          const uint32_t dst = (which ? tDO : tQ) + lane_off + ch * (D / 4);
          if constexpr (D == 128) tmem_st32(dst, w);
          else tmem_st16(dst, w);
        }
      }
      tc_wait_st();
      tc_fence_before();
      warp_arrive(bar_qt_ready);
      warp_arrive(bar_qdo_empty);
      for (int i = 0; i < n; ++i, ++T) {
        // ---- P(T): registers only
        ok = mbar_wait(bar_s_full, T & 1, ab, WAIT_DQ_S);
        if (!ok) break;
        tc_fence_after();
        float pr[64];
        {
          uint32_t sv[64];
          tmem_ld32(tS + lane_off + ch * 64, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
          tmem_ld32(tS + lane_off + ch * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
          tc_wait_ld();
          tc_fence_before();
          warp_arrive(bar_s_read);
          // number of leading key columns of this tile that the row sees
          const int limit = (i < nA) ? (a_len - i * 128) : (q_pos0 + r + 1 - (i - nA) * 128);
          const int lim = limit - ch * 64;
          // packed fp32 for the scale-and-subtract; the pairs kDqFmaMask names take exp2 on the FMA pipe
          const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nl2 = make_float2(nlse2, nlse2);
#pragma unroll
          for (int c = 0; c < 64; c += 2) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1])), sc2, nl2);
            const float2 e = ((kDqFmaMask >> ((c / 2) & 15)) & 1) ? ex2_fma2(x) : ex2_2(x);
            pr[c] = e.x; pr[c + 1] = e.y;
          }
          if (lim < 64) {
#pragma unroll
            for (int c = 0; c < 64; ++c)
              if (c >= lim) pr[c] = 0.f;
          }
        }
        // ---- dS(T) = P * (scale*dP - scale*delta), bf16 over dP
        ok = mbar_wait(bar_dp_full, T & 1, ab, WAIT_DQ_DP);
        if (!ok) break;
        tc_fence_after();
        {
          const float2 sc2 = make_float2(p.scale, p.scale), nd2 = make_float2(ndlt, ndlt);
          uint32_t dpv[64];
          tmem_ld32(tDP + lane_off + ch * 64, *reinterpret_cast<uint32_t(*)[32]>(&dpv[0]));
          tmem_ld32(tDP + lane_off + ch * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&dpv[32]));
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t dd[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float2 t = __ffma2_rn(make_float2(__uint_as_float(dpv[c * 32 + 2 * e]), __uint_as_float(dpv[c * 32 + 2 * e + 1])), sc2, nd2);
              const float2 a = __fmul2_rn(make_float2(pr[c * 32 + 2 * e], pr[c * 32 + 2 * e + 1]), t);
              dd[e] = pack_bf16(a.x, a.y);
            }
            tmem_st16(tDP + lane_off + ch * 64 + c * 16, dd);
          }
        }
        tc_wait_st();
        tc_fence_before();
        warp_arrive(bar_ds_ready);
      }
      if (!ok) break;
      // ---- epilogue: dQ row r, columns (D/2)*ch .., rounded to bf16 once
      ok = mbar_wait(bar_dq_full, ic & 1, ab, WAIT_DQ_FULL);
      if (!ok) break;
      tc_fence_after();
      {
        constexpr int HALF = D / 2;
        __nv_bfloat16 *dst_row = p.dq + (((long long)q_tok0 + r) * p.h_q + head) * p.d + ch * HALF;
#pragma unroll
        for (int c = 0; c < HALF / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(tDQ + lane_off + ch * HALF + c * 32, v);
          tc_wait_ld();
          if (r < q_rows && p.dq_f32) {
            float4 *dst = reinterpret_cast<float4 *>(p.dq_f32 + (((long long)q_tok0 + r) * p.h_q + head) * p.d + ch * HALF + c * 32);
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (ch * HALF + c * 32 + 4 * e < p.d) dst[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]), __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
          } else if (r < q_rows) {
            uint4 *dst = reinterpret_cast<uint4 *>(dst_row + c * 32);
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (ch * HALF + c * 32 + 8 * e < p.d) dst[e] = make_uint4(pack_bf16(__uint_as_float(v[8 * e]), __uint_as_float(v[8 * e + 1])),
                                  pack_bf16(__uint_as_float(v[8 * e + 2]), __uint_as_float(v[8 * e + 3])),
                                  pack_bf16(__uint_as_float(v[8 * e + 4]), __uint_as_float(v[8 * e + 5])),
                                  pack_bf16(__uint_as_float(v[8 * e + 6]), __uint_as_float(v[8 * e + 7])));
          }
        }
      }
      tc_fence_before();
      warp_arrive(bar_dq_empty);
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
  if (warp == 9) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

}  // namespace augtree
