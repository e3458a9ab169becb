// Backward, key side (dK, dV), KV-stationary: one persistent CTA per replay lane
// walks its list of (KV tile, KV head) items.  An item keeps its K and V tile in
// shared memory and streams past it every query tile that can see it: for a
// prompt-KV tile in replay, all response tiles of all G branches and all query
// heads of the KV head, which is the many-to-one sum of Eq. 2 done in one TMEM
// accumulator in a fixed order by one owner; for a tile inside a sequence, the
// causal query tiles of that sequence.  (The query side, dQ, is computed by
// dq_kernel, query-stationary, so that neither side needs atomics.)
//
// Per (KV tile, Q tile, head) pair T, with S^T = K Q^T so that a TMEM lane is a key:
//   P^T  = exp2(S^T * scale*log2e - lse2[q])          (element-wise warps; packed fp32 arithmetic)
//   dP^T = V dO^T
//   dS^T = P^T * (scale*dP^T - scale*delta[q])        (element-wise warps)
//   dV  += P^T dO      (A = P^T from TMEM)
//   dK  += dS^T Q      (A = dS^T from TMEM)
//
// Warp roles (576 threads): warps 0-15 element-wise (warp w: TMEM lanes
// 32*(w%4).., query columns 32*(w/4)..), warp 16 lane 0 TMA loads, warp 17 MMA
// issue (whole warp in lockstep, one elected lane).  TMEM columns: R0 [0,128) S^T, overwritten in place by P^T (bf16);
// R1 [128,256) dP^T, overwritten in place by dS^T (bf16); dV at 256; dK at 256 + D.
// MMA issue order in steady state: dP(T), dV(T), S(T+1), dK(T); the tensor pipe
// executes in order, so S(T+1) may overwrite R0 once dV(T) is issued and
// dP(T+1) may overwrite R1 once dK(T) is issued.
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace augtree {

struct BwdParams {
  const int32_t *items;     // lane order, 8 ints each
  const int32_t *lane_ptr;  // [gridDim.x + 1]
  const int32_t *segs;      // [n_seg][3] {first query token, length, first tile index}
  const float *stats;       // [h_q][n_tiles][2][128]: -lse*log2e (-inf past the end), -scale*rowsum(dO*O)
  __nv_bfloat16 *dk_out, *dv_out;  // mode-0 items when causal_fp32 == 0: [kv tokens, h_kv, D] bf16
  float *dk_acc, *dv_acc;   // fp32 [prompt tokens, h_kv, D]: mode-1 items, and mode-0 items when causal_fp32 != 0
  long long n_tiles;        // query tiles in the stats table
  int h_q, h_kv;
  int d;                    // head dimension of the tensors (<= D; columns d.. of every tile read as zero)
  int causal_fp32;
  float scale, scale_log2;
  int *status;
  long long wait_budget;    // clocks a wait may take before the kernel gives up
  int kind;                 // schedule index: status[2 + kind] counts finished items
  int test_flags;           // TEST_SKIP_BWD_LOAD: lane 0 never loads the first dO tile of its first item
  int no_own;               // partial-state variant: items inside a sequence (mode 0) are skipped by every role
  // dS hand-off (null: off): dS^T of every (KV tile, query tile, head) pair is also stored, bf16, as a row-major
  // [128 keys][128 queries] tile in slot pair_tab[t].x * h_q + head * pair_tab[t].y + (index of the KV tile among
  // those the query tile sees), for a query-side kernel that then needs neither S nor dP again (dql_kernel)
  __nv_bfloat16 *ds_out;
  const int4 *pair_tab;     // per query tile {first slot / h_q, KV tiles seen, prompt KV tiles among them, 0}
};

constexpr int kBwdThreads = 576;  // 16 element-wise warps, TMA warp, MMA warp
#ifndef AUGTREE_BWD_FMA_MASK
#define AUGTREE_BWD_FMA_MASK 0x8888u
#endif
constexpr uint32_t kBwdFmaMask = AUGTREE_BWD_FMA_MASK;  // pairs (of a thread's 16) whose exp2 runs on the FMA pipe

template <int D>
struct BwdSmem {
  static constexpr int kStages = 2;
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kOffK = 0, kOffV = kTileBytes;
  static constexpr int kOffQ = 2 * kTileBytes;                     // [kStages]
  static constexpr int kOffDo = kOffQ + kStages * kTileBytes;      // [kStages]
  static constexpr int kOffStats = kOffDo + kStages * kTileBytes;  // [kStages][2][128] floats
  static constexpr int kOffBar = kOffStats + kStages * 1024;
  static constexpr int kBytes = kOffBar + 256;
};

// bulk copy global -> shared (1-D), completion on an mbarrier
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
           const __grid_constant__ CUtensorMap tm_k0, const __grid_constant__ CUtensorMap tm_v0,
           const __grid_constant__ CUtensorMap tm_k1, const __grid_constant__ CUtensorMap tm_v1, const BwdParams p) {
  using SM = BwdSmem<D>;
  constexpr int TILE = SM::kTileBytes;
  constexpr int NBOX = D / 64;
  constexpr int NST = SM::kStages;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {  // the 128-byte swizzle needs 1024-byte aligned tiles
    if (threadIdx.x == 0 && atomicCAS(p.status, 0, -6) == 0) p.status[1] = 1;
    return;
  }
  const uint32_t sK = base + SM::kOffK, sV = base + SM::kOffV, sQ0 = base + SM::kOffQ, sDo0 = base + SM::kOffDo;
  const uint32_t sStats0 = base + SM::kOffStats;
  const uint32_t bars = base + SM::kOffBar;
  const uint32_t bar_kv_full = bars, bar_kv_empty = bars + 8;
  const uint32_t bar_q_full = bars + 16, bar_q_empty = bars + 48;     // [NST <= 4] each
  const uint32_t bar_do_full = bars + 80, bar_do_empty = bars + 112;  // [NST <= 4] each
  const uint32_t bar_s_full = bars + 144, bar_p_ready = bars + 152, bar_dp_full = bars + 160, bar_ds_ready = bars + 168;
  const uint32_t bar_acc_full = bars + 176, bar_acc_empty = bars + 184, bar_p_hi = bars + 208;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_raw + SM::kOffBar + 192);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + SM::kOffBar + 200);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar_kv_full, 1); mbar_init(bar_kv_empty, 1);
    for (int s = 0; s < NST; ++s) {
      mbar_init(bar_q_full + 8 * s, 1); mbar_init(bar_q_empty + 8 * s, 1);
      mbar_init(bar_do_full + 8 * s, 1); mbar_init(bar_do_empty + 8 * s, 1);
    }
    mbar_init(bar_s_full, 1); mbar_init(bar_p_ready, 16); mbar_init(bar_p_hi, 16); mbar_init(bar_dp_full, 1); mbar_init(bar_ds_ready, 16);
    mbar_init(bar_acc_full, 1); mbar_init(bar_acc_empty, 16);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 17) { tmem_alloc(smem_u32((const void *)tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tR0 = tmem, tR1 = tmem + 128, tDV = tmem + 256, tDK = tmem + 256 + D;
  const AbortCtx ab{abort_flag, p.status, p.wait_budget};
  const int rep = p.h_q / p.h_kv;
  const int it_begin = p.lane_ptr[blockIdx.x], it_end = p.lane_ptr[blockIdx.x + 1];

  if (warp == 16) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_do); tma_prefetch_desc(&tm_k0);
      tma_prefetch_desc(&tm_v0); tma_prefetch_desc(&tm_k1); tma_prefetch_desc(&tm_v1);
      uint32_t ic = 0, T = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const int32_t *I = p.items + (size_t)it * 8;
        const int kv_tok0 = I[0], kv_pos0 = I[1], kvh = I[3], mode = I[4], seg0 = I[5], nseg = I[6];
        if (p.no_own && mode == 0) continue;
        if (ic > 0) {
          ok = mbar_wait(bar_kv_empty, (ic - 1) & 1, ab, WAIT_BWD_KV_EMPTY);
          if (!ok) break;
        }
        mbar_expect_tx(bar_kv_full, 2 * TILE);
        for (int b = 0; b < NBOX; ++b) {
          tma_load_3d(sK + b * 16384, mode ? &tm_k1 : &tm_k0, bar_kv_full, b * 64, kvh, kv_tok0);
          tma_load_3d(sV + b * 16384, mode ? &tm_v1 : &tm_v0, bar_kv_full, b * 64, kvh, kv_tok0);
        }
        for (int sg = seg0; sg < seg0 + nseg && ok; ++sg) {
          const int s_tok0 = p.segs[3 * sg], s_len = p.segs[3 * sg + 1], s_tile0 = p.segs[3 * sg + 2];
          const int nqt = (s_len + 127) >> 7;
          for (int qt = mode ? 0 : (kv_pos0 >> 7); qt < nqt && ok; ++qt)
            for (int j = 0; j < rep; ++j, ++T) {
              const uint32_t st = T % NST, par = ((T / NST) & 1) ^ 1;
              const int head = kvh * rep + j, row = s_tok0 + qt * 128;
              ok = mbar_wait(bar_q_empty + 8 * st, par, ab, WAIT_BWD_QDO_EMPTY);
              if (!ok) break;
              mbar_expect_tx(bar_q_full + 8 * st, TILE + 1024);
              for (int b = 0; b < NBOX; ++b) tma_load_3d(sQ0 + st * TILE + b * 16384, &tm_q, bar_q_full + 8 * st, b * 64, head, row);
              bulk_load_1d(sStats0 + st * 1024, p.stats + ((long long)head * p.n_tiles + s_tile0 + qt) * 256, 1024,
                           bar_q_full + 8 * st);
              if ((p.test_flags & TEST_SKIP_BWD_LOAD) && blockIdx.x == 0 && T == 0) continue;  // injected fault
              ok = mbar_wait(bar_do_empty + 8 * st, par, ab, WAIT_BWD_QDO_EMPTY);
              if (!ok) break;
              mbar_expect_tx(bar_do_full + 8 * st, TILE);
              for (int b = 0; b < NBOX; ++b) tma_load_3d(sDo0 + st * TILE + b * 16384, &tm_do, bar_do_full + 8 * st, b * 64, head, row);
            }
        }
        ++ic;
      }
    }
  } else if (warp == 17) {
    // -------------------------------------------------------------- MMA issuer
    // The whole warp runs the loops in lockstep and one elected lane issues (warp-uniform descriptor
    // arithmetic: few instructions per MMA, which matters next to two busy element-wise warps on the same
    // scheduler).  Each group looks at the barrier of the group after it before its own last two MMAs
    // (`have`), so that a hand-off which has already happened costs the tensor pipe nothing.
    {
      constexpr uint32_t IDESC_ST = make_idesc(128, 128, 0, 0);  // S^T, dP^T: both operands K-major
      constexpr uint32_t IDESC_ACC = make_idesc(128, D, 0, 1);   // dV, dK: A from TMEM, B = dO / Q MN-major
      constexpr int NK = D / 16;
      const bool elected = elect_one();
      const int it_b = __shfl_sync(0xffffffffu, it_begin, 0), it_e = __shfl_sync(0xffffffffu, it_end, 0);
      uint32_t ic = 0, T = 0;
      bool ok = true;
      const uint32_t kk_lo = sdesc_lo(sK, 16), vk_lo = sdesc_lo(sV, 16);
      auto need = [&](bool have, uint32_t bar, uint32_t par, int site) -> bool {
        if (!have && !mbar_wait(bar, par, ab, site)) return false;
        tc_fence_after();
        return true;
      };
      for (int it = it_b; it < it_e && ok; ++it) {
        const int32_t *I = p.items + (size_t)it * 8;
        const int kv_pos0 = I[1], mode = I[4], seg0 = I[5], nseg = I[6];
        if (p.no_own && __shfl_sync(0xffffffffu, mode, 0) == 0) continue;
        int n_pairs = 0;
        for (int sg = seg0; sg < seg0 + nseg; ++sg) {
          const int nqt = (p.segs[3 * sg + 1] + 127) >> 7;
          n_pairs += (nqt - (mode ? 0 : (kv_pos0 >> 7))) * rep;
        }
        n_pairs = __shfl_sync(0xffffffffu, n_pairs, 0);
        ok = mbar_wait(bar_kv_full, ic & 1, ab, WAIT_BWD_KV_FULL);
        if (!ok) break;
        bool have_do = false;
        {  // prologue: S^T of the item's first pair -> R0
          const uint32_t st = T % NST, par = (T / NST) & 1;
          ok = need(false, bar_q_full + 8 * st, par, WAIT_BWD_QDO_FULL);
          if (!ok) break;
          const uint32_t qk_lo = sdesc_lo(sQ0 + st * TILE, 16);
          mma_group<NK>(elected,
                        [&](int k) { mma_ss2(tR0, kk_lo + kstep_kmajor(k), qk_lo + kstep_kmajor(k), IDESC_ST, k > 0); },
                        [&]() { have_do = mbar_test(bar_do_full + 8 * st, par); });
          if (elected) tc_commit(bar_s_full);
        }
        for (int i = 0; i < n_pairs && ok; ++i, ++T) {
          const uint32_t st = T % NST, par = (T / NST) & 1;
          const uint32_t st1 = (T + 1) % NST, par1 = ((T + 1) / NST) & 1;
          const bool more = i + 1 < n_pairs;
          const uint32_t dok_lo = sdesc_lo(sDo0 + st * TILE, 16), dom_lo = sdesc_lo(sDo0 + st * TILE, 16384);
          const uint32_t qm_lo = sdesc_lo(sQ0 + st * TILE, 16384), qk1_lo = sdesc_lo(sQ0 + st1 * TILE, 16);
          const uint32_t acc0 = i > 0 ? 1u : 0u;
          bool have_p = false, have_q = false, have_ds = false;
          // ---- dP^T(T) = V dO^T -> R1
          ok = need(have_do, bar_do_full + 8 * st, par, WAIT_BWD_QDO_FULL);
          if (!ok) break;
          mma_group<NK>(elected,
                        [&](int k) { mma_ss2(tR1, vk_lo + kstep_kmajor(k), dok_lo + kstep_kmajor(k), IDESC_ST, k > 0); },
                        [&]() { have_p = mbar_test(bar_p_ready, T & 1); });
          if (elected) tc_commit(bar_dp_full);
          // ---- dV += P^T(T) dO(T)
          if (i == 0 && ic > 0) {  // the previous item's dV/dK must have left TMEM
            ok = mbar_wait(bar_acc_empty, (ic - 1) & 1, ab, WAIT_BWD_ACC_EMPTY);
            if (!ok) break;
          }
          ok = need(have_p, bar_p_ready, T & 1, WAIT_BWD_PDS_FULL);
          if (!ok) break;
          // (query columns 16k..16k+15: P^T sits at R0 columns 32 (k / 2) + 8 (k % 2), over its own thread's S^T.)
          // Every element-wise warp hands over the first 16 of its 32 query columns (the even k steps) while it is
          // still exponentiating the rest, so half of this GEMM runs under the second half of the P phase: the loop
          // dV(T) -> S(T+1) -> P(T+1) -> dV(T+1) is what bounds a pair.
          bool have_hi = false;
          mma_group<4>(elected,
                       [&](int k) { mma_ts2(tDV, tR0 + 32 * k, dom_lo + kstep_mnmajor(2 * k), IDESC_ACC, acc0 | (uint32_t)(k > 0)); },
                       [&]() { have_hi = mbar_test(bar_p_hi, T & 1); });
          ok = need(have_hi, bar_p_hi, T & 1, WAIT_BWD_PDS_FULL);
          if (!ok) break;
          mma_group<4>(elected,
                       [&](int k) { mma_ts2(tDV, tR0 + 32 * k + 8, dom_lo + kstep_mnmajor(2 * k + 1), IDESC_ACC, 1u); },
                       [&]() { have_q = more && mbar_test(bar_q_full + 8 * st1, par1); });
          if (elected) tc_commit(bar_do_empty + 8 * st);
          // ---- S^T(T+1) = K Q^T -> R0 (free: dV(T) was issued and the tensor pipe runs in order)
          if (more) {
            ok = need(have_q, bar_q_full + 8 * st1, par1, WAIT_BWD_QDO_FULL);
            if (!ok) break;
            mma_group<NK>(elected,
                          [&](int k) { mma_ss2(tR0, kk_lo + kstep_kmajor(k), qk1_lo + kstep_kmajor(k), IDESC_ST, k > 0); },
                          [&]() { have_ds = mbar_test(bar_ds_ready, T & 1); });
            if (elected) tc_commit(bar_s_full);
          }
          // ---- dK += dS^T(T) Q(T)
          ok = need(have_ds, bar_ds_ready, T & 1, WAIT_BWD_PDS_FULL);
          if (!ok) break;
          have_do = false;
          mma_group<8>(elected,
                       [&](int k) {
                         mma_ts2(tDK, tR1 + 32 * (k >> 1) + 8 * (k & 1), qm_lo + kstep_mnmajor(k), IDESC_ACC, acc0 | (uint32_t)(k > 0));
                       },
                       [&]() { have_do = more && mbar_test(bar_do_full + 8 * st1, par1); });
          if (elected) tc_commit(bar_q_empty + 8 * st);
        }
        if (!ok) break;
        if (elected) { tc_commit(bar_acc_full); tc_commit(bar_kv_empty); }
        ++ic;
      }
    }
  } else {
    // ------------------------------------------------------- element-wise warps 0-15
    // Warp w: TMEM lanes (key rows) 32 (w % 4) .., query columns 32 (w / 4) .. of every tile: four threads per
    // key row.  The phases are bound by the latency of their loads and special-function results, which four
    // warps per scheduler hide better than two.
    const int lg = warp & 3, ch = warp >> 2;
    const int r = lg * 32 + lane;  // TMEM lane = key row
    const uint32_t lane_off = (uint32_t)(lg * 32) << 16;
    uint32_t ic = 0, T = 0;
    bool ok = true;
    float pr[32];  // P^T of the current pair: key r, query columns 32*ch .. 32*ch+31

    // P^T(Tn) from S^T(Tn): wait, load, exponentiate, store bf16 over S^T, signal
    auto make_p = [&](uint32_t Tn, int q_base, int kv_pos0, int mode, bool key_valid) -> bool {
      const uint32_t st = Tn % NST;
      if (!mbar_wait(bar_q_full + 8 * st, (Tn / NST) & 1, ab, WAIT_BWD_QDO_FULL)) return false;  // row statistics landed
      if (!mbar_wait(bar_s_full, Tn & 1, ab, WAIT_BWD_S_FULL)) return false;
      tc_fence_after();
      const float *lse2 = reinterpret_cast<const float *>(smem_raw + SM::kOffStats + st * 1024) + ch * 32;
      // query column (inside the tile) from which this key is visible
      const int lo = mode ? 0 : (kv_pos0 + r - q_base);
      const bool all_visible = key_valid && lo <= ch * 32;
      uint32_t sv[32];
      tmem_ld32(tR0 + lane_off + ch * 32, sv);
      tc_wait_ld();
      // packed fp32: one fma per pair for the scale-and-subtract (the table holds -lse*log2e), and the pairs
      // that kBwdFmaMask names take their exp2 on the FMA pipe.  Two halves of 16 query columns, each handed
      // to the MMA warp as soon as it is in TMEM.
      const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int i = 16 * h; i < 16 * h + 16; i += 4) {
          const float4 l4 = *reinterpret_cast<const float4 *>(lse2 + i);
          const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(sv[i + 0]), __uint_as_float(sv[i + 1])), sc2, make_float2(l4.x, l4.y));
          const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3])), sc2, make_float2(l4.z, l4.w));
          const float2 p0 = ((kBwdFmaMask >> (i / 2)) & 1) ? ex2_fma2(x0) : ex2_2(x0);
          const float2 p1 = ((kBwdFmaMask >> (i / 2 + 1)) & 1) ? ex2_fma2(x1) : ex2_2(x1);
          pr[i + 0] = p0.x; pr[i + 1] = p0.y; pr[i + 2] = p1.x; pr[i + 3] = p1.y;
        }
        if (!all_visible) {
#pragma unroll
          for (int i = 16 * h; i < 16 * h + 16; ++i)
            if (!key_valid || ch * 32 + i < lo) pr[i] = 0.f;
        }
        uint32_t pk[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) pk[i] = pack_bf16(pr[16 * h + 2 * i], pr[16 * h + 2 * i + 1]);
        tmem_st8(tR0 + lane_off + ch * 32 + 8 * h, pk);
        tc_wait_st();
        tc_fence_before();
        warp_arrive(h ? bar_p_hi : bar_p_ready);
      }
      return true;
    };

    for (int it = it_begin; it < it_end && ok; ++it) {
      const int32_t *I = p.items + (size_t)it * 8;
      const int kv_tok0 = I[0], kv_pos0 = I[1], kv_rows = I[2], kvh = I[3], mode = I[4], seg0 = I[5], nseg = I[6];
      if (p.no_own && mode == 0) continue;
      const bool key_valid = r < kv_rows;
      bool first = true;
      for (int sg = seg0; sg < seg0 + nseg && ok; ++sg) {
        const int s_len = p.segs[3 * sg + 1], s_tile0 = p.segs[3 * sg + 2];
        const int nqt = (s_len + 127) >> 7;
        const int qt0 = mode ? 0 : (kv_pos0 >> 7);
        for (int qt = qt0; qt < nqt && ok; ++qt) {
          // hand-off: where this thread's 64 bytes of the pair's dS^T tile go (head j = 0), and the step to the next head
          __nv_bfloat16 *ds_dst = nullptr;
          long long ds_step = 0;
          if (p.ds_out) {
            const int4 pt = __ldg(p.pair_tab + s_tile0 + qt);
            const long long slot = (long long)pt.x * p.h_q + (long long)(kvh * rep) * pt.y + (mode ? 0 : pt.z) + (kv_pos0 >> 7);
            ds_dst = p.ds_out + slot * 16384 + r * 128 + ch * 32;
            ds_step = (long long)pt.y * 16384;
          }
          for (int j = 0; j < rep; ++j, ++T, ds_dst += ds_step) {
            const uint32_t st = T % NST;
            if (first) {  // the item's first pair has no predecessor to pipeline behind
              ok = make_p(T, qt * 128, kv_pos0, mode, key_valid);
              if (!ok) break;
              first = false;
            }
            // ---- dS^T(T) = P^T * (scale*dP^T - scale*delta), bf16 over dP^T in R1
            ok = mbar_wait(bar_dp_full, T & 1, ab, WAIT_BWD_S_FULL);
            if (!ok) break;
            tc_fence_after();
            {
              const float *dl = reinterpret_cast<const float *>(smem_raw + SM::kOffStats + st * 1024) + 128 + ch * 32;
              uint32_t dpv[32];
              tmem_ld32(tR1 + lane_off + ch * 32, dpv);
              tc_wait_ld();
              uint32_t dd[16];
              const float2 sc2 = make_float2(p.scale, p.scale);
#pragma unroll
              for (int i = 0; i < 32; i += 4) {
                const float4 d4 = *reinterpret_cast<const float4 *>(dl + i);   // -scale * delta
                const float2 t0 = __ffma2_rn(make_float2(__uint_as_float(dpv[i + 0]), __uint_as_float(dpv[i + 1])), sc2, make_float2(d4.x, d4.y));
                const float2 t1 = __ffma2_rn(make_float2(__uint_as_float(dpv[i + 2]), __uint_as_float(dpv[i + 3])), sc2, make_float2(d4.z, d4.w));
                const float2 a0 = __fmul2_rn(make_float2(pr[i + 0], pr[i + 1]), t0);
                const float2 a1 = __fmul2_rn(make_float2(pr[i + 2], pr[i + 3]), t1);
                dd[i / 2] = pack_bf16(a0.x, a0.y);
                dd[i / 2 + 1] = pack_bf16(a1.x, a1.y);
              }
              tmem_st16(tR1 + lane_off + ch * 32, dd);
              if (p.ds_out) {
                // hand-off: this thread's 32 values are 64 contiguous bytes of the stored tile, written as two whole
                // 32-byte sectors (16-byte stores leave half sectors behind and were measured 1.7x slower)
#pragma unroll
                for (int i = 0; i < 2; ++i) st_global_v8(ds_dst + 16 * i, dd + 8 * i);
              }
            }
            tc_wait_st();
            tc_fence_before();
            warp_arrive(bar_ds_ready);
            // ---- P^T(T+1), if the item has another pair (same iteration order as the other roles)
            {
              int qt2 = qt, j2 = j + 1;
              bool more = true;
              if (j2 == rep) { j2 = 0; ++qt2; }
              int q_base2 = qt2 * 128;
              if (qt2 >= nqt) {
                if (sg + 1 < seg0 + nseg) q_base2 = qt0 * 128; else more = false;
              }
              if (more) {
                ok = make_p(T + 1, q_base2, kv_pos0, mode, key_valid);
                if (!ok) break;
              }
            }
          }
        }
      }
      if (!ok) break;
      // ---- item epilogue: dV, dK of key row r, columns (D/4)*ch ..
      ok = mbar_wait(bar_acc_full, ic & 1, ab, WAIT_BWD_ACC_FULL);
      if (!ok) break;
      tc_fence_after();
      const long long krow = ((long long)kv_tok0 + r) * p.h_kv + kvh;
      const bool to_fp32 = mode || p.causal_fp32;
      constexpr int QUART = D / 4;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        const int col0 = ch * QUART;
        uint32_t v[QUART];
        if constexpr (D == 128) tmem_ld32((which ? tDK : tDV) + lane_off + col0, v);
        else tmem_ld16((which ? tDK : tDV) + lane_off + col0, v);
        tc_wait_ld();
        if (key_valid) {
          if (to_fp32) {
            float4 *dst = reinterpret_cast<float4 *>((which ? p.dk_acc : p.dv_acc) + krow * p.d + col0);
#pragma unroll
            for (int i = 0; i < QUART / 4; ++i) {
              if (col0 + 4 * i >= p.d) break;  // padding columns
              float4 a = dst[i];
              a.x += __uint_as_float(v[4 * i]); a.y += __uint_as_float(v[4 * i + 1]);
              a.z += __uint_as_float(v[4 * i + 2]); a.w += __uint_as_float(v[4 * i + 3]);
              dst[i] = a;
            }
          } else {
            uint4 *dst = reinterpret_cast<uint4 *>((which ? p.dk_out : p.dv_out) + krow * p.d + col0);
#pragma unroll
            for (int i = 0; i < QUART / 8; ++i)
              if (col0 + 8 * i < p.d) dst[i] = make_uint4(pack_bf16(__uint_as_float(v[8 * i]), __uint_as_float(v[8 * i + 1])),
                                  pack_bf16(__uint_as_float(v[8 * i + 2]), __uint_as_float(v[8 * i + 3])),
                                  pack_bf16(__uint_as_float(v[8 * i + 4]), __uint_as_float(v[8 * i + 5])),
                                  pack_bf16(__uint_as_float(v[8 * i + 6]), __uint_as_float(v[8 * i + 7])));
          }
        }
      }
      tc_fence_before();
      warp_arrive(bar_acc_empty);
      if (warp == 0 && lane == 0) atomicAdd(p.status + 2 + p.kind, 1);  // item finished (work accounting)
      ++ic;
    }
  }

  __syncwarp();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) {}
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 17) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// Row statistics of the backward pass, stored per 128-row query tile, negated so that the tile kernels
// fold them in with one fused multiply-add:
// stats[head][tile][0][i] = -lse * log2(e) (-inf for rows past the tile's end: their P becomes 0),
// stats[head][tile][1][i] = -scale * sum_d dO * O (0 past the end).  One warp per 16 rows.
template <int D>
__global__ void bwd_preprocess_kernel(const __nv_bfloat16 *o, const __nv_bfloat16 *d_o, const float *lse, const int32_t *tiles,
                                      float *stats, long long n_tok, long long n_tiles, int h_q, int d, float scale) {
  const int tile = blockIdx.x, head = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tok0 = tiles[2 * tile], rows = tiles[2 * tile + 1];
  float *out = stats + ((long long)head * n_tiles + tile) * 256;
  // a lane reads 16 bytes of a row: D / 8 lanes per row, 32 / (D / 8) rows per warp pass; a warp owns 16 rows and
  // issues the loads of all its passes before it reduces any (HBM-bound: keep many loads in flight)
  constexpr int LPR = D / 8, RPP = 32 / LPR, PASSES = 16 / RPP;
  const int sub = lane / LPR, part = lane % LPR;
  uint4 vo[PASSES], vd[PASSES];
#pragma unroll
  for (int ps = 0; ps < PASSES; ++ps) {
    const int i = warp * 16 + ps * RPP + sub;
    vo[ps] = make_uint4(0, 0, 0, 0); vd[ps] = make_uint4(0, 0, 0, 0);
    if (i < rows && part * 8 < d) {
      const long long w = (((long long)tok0 + i) * h_q + head) * d + part * 8;
      vo[ps] = *reinterpret_cast<const uint4 *>(o + w);
      vd[ps] = *reinterpret_cast<const uint4 *>(d_o + w);
    }
  }
#pragma unroll
  for (int ps = 0; ps < PASSES; ++ps) {
    const int i = warp * 16 + ps * RPP + sub;
    const uint32_t a[4] = {vo[ps].x, vo[ps].y, vo[ps].z, vo[ps].w}, b[4] = {vd[ps].x, vd[ps].y, vd[ps].z, vd[ps].w};
    float acc = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&a[e]));
      const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b[e]));
      acc = fmaf(x.x, y.x, fmaf(x.y, y.y, acc));
    }
#pragma unroll
    for (int sft = LPR / 2; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
    if (part == 0) {
      const bool valid = i < rows;
      out[i] = valid ? -lse[(long long)head * n_tok + tok0 + i] * 1.4426950408889634f : -INFINITY;
      out[128 + i] = valid ? -acc * scale : 0.f;
    }
  }
}

// fp32 -> bf16 (optional bf16 copies of the prompt gradients)
__global__ void cast_bf16_kernel(const float *src, __nv_bfloat16 *dst, long long n4) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float4 v = reinterpret_cast<const float4 *>(src)[i];
  uint2 w;
  w.x = pack_bf16(v.x, v.y);
  w.y = pack_bf16(v.z, v.w);
  reinterpret_cast<uint2 *>(dst)[i] = w;
}

}  // namespace augtree
