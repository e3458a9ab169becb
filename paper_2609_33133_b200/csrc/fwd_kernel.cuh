// Forward tile kernel: one persistent CTA per replay lane walks its list of
// (pair of query tiles, head) items.  An item's keys are an unmasked range of the
// shared prompt KV followed by a causal range of the query's own sequence
// (Eq. 1); the online-softmax state (m, l, O_acc) of Sec. 3.3 is carried across
// all of the item's KV tiles, which merges the two parts' partial states as it
// goes.  The two query tiles of an item share every K/V tile the CTA loads.
//
// Warp roles (320 threads): warps 0-7 are the softmax warps, warp 8 lane 0 issues
// TMA loads, warp 9 issues tcgen05 MMAs (whole warp in lockstep, one elected lane).
// All eight softmax warps work on ONE query tile at a time, 16 rows each, and
// alternate between the two tiles.  They read S in the accumulator-fragment layout
// (tcgen05.ld 16x256b): a row is spread over the four threads of a quad, so the row
// maximum and sum are two shuffles and no warp waits for another.  What bounds a KV
// step is the loop  softmax_g -> PV_g -> S_g(next) -> softmax_g  of one tile, so the
// softmax of a tile has to be short; the other tile's MMAs run under it.
// TMEM: S/P of tile 0 at column 0, of tile 1 at 128; O of tile 0 at 256, of tile 1 at 384.
// MMA issue order per KV tile j: PV0(j), S0(j+1), PV1(j), S1(j+1).
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace augtree {

struct FwdParams {
  const int32_t *items;     // lane order, 12 ints each
  const int32_t *lane_ptr;  // [gridDim.x + 1]
  __nv_bfloat16 *o;         // [tokens, h_q, D]
  float *lse;               // [h_q, tokens]
  float *part_o;            // [splits, tokens, h_q, D] fp32 (normalised partial outputs)
  float *part_lse;          // [splits, h_q, tokens]
  long long n_tok;          // tokens in the query tensor
  int h_q;
  int d;                    // head dimension of the tensors (<= D; D is the padded tile width, columns d.. read as zero)
  float scale_log2;         // softmax scale * log2(e)
  const float *kmax2;       // [h_kv] largest squared key norm of the call's K tensors (key_norm_kernel)
  int *status;
  long long wait_budget;    // clocks a wait may take before the kernel gives up
  int kind;                 // schedule index: status[2 + kind] counts finished items
  int test_flags;           // TEST_SKIP_FWD_LOAD: lane 0 never loads the first V tile of its first item
  int state_mode;           // STATE_OUT | STATE_NO_OWN: partial-state variant for context-parallel replay (below)
};

// Partial-state variant (Sec. 3.3, "Common tile semantics": a query block against one KV shard gives a partial
// state; the states along a query's row are merged afterwards).  STATE_OUT: every item writes its normalised fp32
// output and its LSE into part_o / part_lse (shard slot 0) instead of the final tensors.  STATE_NO_OWN: the causal
// range of the query's own sequence is left out, so that the state covers the plan's prompt keys alone.
enum : int { STATE_OUT = 1, STATE_NO_OWN = 2 };

constexpr int kFwdThreads = 320;
constexpr float kRescaleThreshold = 8.0f;  // log2 units: P stays <= 2^8 while the row maximum is tracked
// When |q_a| max_b |k_b| scale log2(e) (a bound on every score of row a, by Cauchy-Schwarz) is less than this many
// log2 units above the row's maximum over its first KV tile, no later exponential can exceed 2^60: with fp32
// accumulators and bf16's fp32-sized exponent nothing overflows and nothing loses precision (softmax does not
// depend on the reference), so the row maximum of the later tiles is not computed at all.
constexpr float kSkipMaxHeadroom = 60.0f;
#ifndef AUGTREE_FWD_FMA_MASK
#define AUGTREE_FWD_FMA_MASK 0x8888u
#endif
constexpr uint32_t kFwdFmaMask = AUGTREE_FWD_FMA_MASK;  // column blocks (of 16) whose exp2 runs on the FMA pipe

template <int D>
struct FwdSmem {
  static constexpr int kStages = 4;  // K/V ring slots
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kOffQ = 0;                       // two query tiles
  static constexpr int kOffKV = 2 * kTileBytes;         // [kStages]
  static constexpr int kOffBar = kOffKV + kStages * kTileBytes;
  static constexpr int kBytes = kOffBar + 256;
};

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_ka,
           const __grid_constant__ CUtensorMap tm_va, const __grid_constant__ CUtensorMap tm_kb,
           const __grid_constant__ CUtensorMap tm_vb, const FwdParams p) {
  using SM = FwdSmem<D>;
  constexpr int TILE = SM::kTileBytes;
  constexpr int NBOX = D / 64;
  constexpr int NS = SM::kStages;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {  // the 128-byte swizzle needs 1024-byte aligned tiles
    if (threadIdx.x == 0 && atomicCAS(p.status, 0, -6) == 0) p.status[1] = 3;
    return;
  }
  const uint32_t sQ = base + SM::kOffQ, sKV = base + SM::kOffKV;
  const uint32_t bars = base + SM::kOffBar;
  const uint32_t bar_q_full = bars, bar_q_empty = bars + 8;
  const uint32_t bar_kv_full = bars + 16, bar_kv_empty = bars + 48;  // [NS <= 4] each
  const uint32_t bar_s_full = bars + 80, bar_p_full = bars + 96;     // [2] each: per query tile
  const uint32_t bar_o_full = bars + 112, bar_o_empty = bars + 128;  // [2] each
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_raw + SM::kOffBar + 144);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + SM::kOffBar + 152);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar_q_full, 1); mbar_init(bar_q_empty, 1 + 8);  // Q slot free: last S MMA of the item done, 8 warps read their rows
    for (int s = 0; s < NS; ++s) { mbar_init(bar_kv_full + 8 * s, 1); mbar_init(bar_kv_empty + 8 * s, 1); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(bar_s_full + 8 * g, 1); mbar_init(bar_p_full + 8 * g, 8);
      mbar_init(bar_o_full + 8 * g, 1); mbar_init(bar_o_empty + 8 * g, 8);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 9) { tmem_alloc(smem_u32((const void *)tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const AbortCtx ab{abort_flag, p.status, p.wait_budget};
  const int it_begin = p.lane_ptr[blockIdx.x], it_end = p.lane_ptr[blockIdx.x + 1];

  if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_ka); tma_prefetch_desc(&tm_va);
      tma_prefetch_desc(&tm_kb); tma_prefetch_desc(&tm_vb);
      uint32_t kvc = 0, ic = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
        const int32_t *I = p.items + (size_t)it * 12;
        const int q_tok0 = I[0], head = I[3], a_tok0 = I[4], a_len = I[5], b_tok0 = I[6], kvh = I[11];
        const int b_len = (p.state_mode & STATE_NO_OWN) ? 0 : I[7];
        const int nA = (a_len + 127) >> 7, n = nA + ((b_len + 127) >> 7);
        ok = mbar_wait(bar_q_empty, (ic & 1) ^ 1, ab, WAIT_FWD_Q_EMPTY);
        if (!ok) break;
        mbar_expect_tx(bar_q_full, 2 * TILE);
        for (int g = 0; g < 2; ++g)
          for (int b = 0; b < NBOX; ++b) tma_load_3d(sQ + g * TILE + b * 16384, &tm_q, bar_q_full, b * 64, head, q_tok0 + g * 128);
        auto load_tile = [&](bool is_v, int j) -> bool {
          const uint32_t slot = kvc % NS, par = ((kvc / NS) & 1) ^ 1;
          if ((p.test_flags & TEST_SKIP_FWD_LOAD) && blockIdx.x == 0 && ic == 0 && is_v && j == 0) { ++kvc; return true; }  // injected fault
          if (!mbar_wait(bar_kv_empty + 8 * slot, par, ab, WAIT_FWD_KV_EMPTY)) return false;
          const bool in_a = j < nA;
          const CUtensorMap *tm = in_a ? (is_v ? &tm_va : &tm_ka) : (is_v ? &tm_vb : &tm_kb);
          const int row = in_a ? a_tok0 + j * 128 : b_tok0 + (j - nA) * 128;
          mbar_expect_tx(bar_kv_full + 8 * slot, TILE);
          for (int b = 0; b < NBOX; ++b)
            tma_load_3d(sKV + slot * TILE + b * 16384, tm, bar_kv_full + 8 * slot, b * 64, kvh, row);
          ++kvc;
          return true;
        };
        // consumption order: K0, then per tile j: V_j, K_{j+1}
        ok = load_tile(false, 0);
        for (int j = 0; j < n && ok; ++j) {
          ok = load_tile(true, j);
          if (ok && j + 1 < n) ok = load_tile(false, j + 1);
        }
      }
    }
  } else if (warp == 9) {
    // -------------------------------------------------------------- MMA issuer
    // The whole warp walks the loops in lockstep and one elected lane issues: all the values that go into
    // the descriptors are then warp-uniform (item fields come through a lane-0 broadcast), which keeps the
    // instruction count per MMA small.  That matters because this warp shares its scheduler with two
    // softmax warps, and a tensor pipe that queues only about two MMAs starves as soon as the issue of the
    // next one is late.
    {
      constexpr uint32_t IDESC_S = make_idesc(128, 128, 0, 0);
      constexpr uint32_t IDESC_PV = make_idesc(128, D, 0, 1);
      const bool elected = elect_one();
      const int it_b = __shfl_sync(0xffffffffu, it_begin, 0), it_e = __shfl_sync(0xffffffffu, it_end, 0);
      uint32_t kvc = 0, ic = 0, T = 0;
      bool ok = true;
      const uint32_t q_lo0 = sdesc_lo(sQ, 16), q_lo1 = sdesc_lo(sQ + TILE, 16);
      // a look that succeeded makes the wait unnecessary (every lane sees the same barrier state)
      auto need = [&](bool have, uint32_t bar, uint32_t par, int site) -> bool {
        if (!have && !mbar_wait(bar, par, ab, site)) return false;
        tc_fence_after();
        return true;
      };
      // K/V tiles of a KV step (V_j and K_{j+1}): waited for at the end of the step before, when this warp
      // would otherwise only be waiting for the next P, so that the path from "P is there" to "PV issued"
      // holds nothing but the P barrier
      uint32_t vslot = 0, kslot = 0;
      bool more = false;
      auto acquire_kv = [&](int j, int n) -> bool {
        vslot = kvc % NS;
        if (!mbar_wait(bar_kv_full + 8 * vslot, (kvc / NS) & 1, ab, WAIT_FWD_KV_FULL)) return false;
        ++kvc;
        more = j + 1 < n;
        if (more) {
          kslot = kvc % NS;
          if (!mbar_wait(bar_kv_full + 8 * kslot, (kvc / NS) & 1, ab, WAIT_FWD_KV_FULL)) return false;
          ++kvc;
        }
        return true;
      };
      for (int it = it_b; it < it_e && ok; ++it, ++ic) {
        const int32_t *I = p.items + (size_t)it * 12;
        const int n = __shfl_sync(0xffffffffu, ((I[5] + 127) >> 7) + ((p.state_mode & STATE_NO_OWN) ? 0 : ((I[7] + 127) >> 7)), 0);
        ok = mbar_wait(bar_q_full, ic & 1, ab, WAIT_FWD_Q_FULL);
        if (!ok) break;
        bool have_p0 = false;
        {  // prologue: S0(0), S1(0)
          const uint32_t slot = kvc % NS;
          ok = need(false, bar_kv_full + 8 * slot, (kvc / NS) & 1, WAIT_FWD_KV_FULL);
          if (!ok) break;
          const uint32_t k_lo = sdesc_lo(sKV + slot * TILE, 16);
          if (elected) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) mma_ss2(tmem, q_lo0 + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
            tc_commit(bar_s_full);
#pragma unroll
            for (int k = 0; k < D / 16; ++k) mma_ss2(tmem + 128, q_lo1 + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
            tc_commit(bar_s_full + 8);
            tc_commit(bar_kv_empty + 8 * slot);
            if (n == 1) tc_commit(bar_q_empty);
          }
          ++kvc;
        }
        ok = acquire_kv(0, n);
        for (int j = 0; j < n && ok; ++j, ++T) {
          const uint32_t v_lo = sdesc_lo(sKV + vslot * TILE, 16384);
          const uint32_t k_lo = sdesc_lo(sKV + kslot * TILE, 16);
          const uint32_t acc0 = j > 0 ? 1u : 0u;
          // ---- query tile 0: PV0(j), then S0(j+1) over P0(j) (the tensor pipe runs in order)
          ok = need(have_p0, bar_p_full, T & 1, WAIT_FWD_P_FULL);
          if (!ok) break;
          if (j == 0 && ic > 0) {
            ok = need(false, bar_o_empty, (ic - 1) & 1, WAIT_FWD_O_EMPTY);
            if (!ok) break;
          }
          if (elected) {
#pragma unroll
            for (int k = 0; k < 8; ++k) mma_ts2(tmem + 256, tmem + k * 8, v_lo + kstep_mnmajor(k), IDESC_PV, acc0 | (uint32_t)(k > 0));
            tc_commit(bar_o_full);
          }
          bool have_p1 = false;
          if (more) {
            if (elected) {
#pragma unroll
              for (int k = 0; k < D / 16 - 2; ++k) mma_ss2(tmem, q_lo0 + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
            }
            have_p1 = mbar_test(bar_p_full + 8, T & 1);
            if (elected) {
#pragma unroll
              for (int k = D / 16 - 2; k < D / 16; ++k) mma_ss2(tmem, q_lo0 + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
              tc_commit(bar_s_full);
            }
          }
          // ---- query tile 1
          ok = need(have_p1, bar_p_full + 8, T & 1, WAIT_FWD_P_FULL);
          if (!ok) break;
          if (j == 0 && ic > 0) {
            ok = need(false, bar_o_empty + 8, (ic - 1) & 1, WAIT_FWD_O_EMPTY);
            if (!ok) break;
          }
          if (elected) {
#pragma unroll
            for (int k = 0; k < 8; ++k) mma_ts2(tmem + 384, tmem + 128 + k * 8, v_lo + kstep_mnmajor(k), IDESC_PV, acc0 | (uint32_t)(k > 0));
            tc_commit(bar_o_full + 8);
            tc_commit(bar_kv_empty + 8 * vslot);
          }
          have_p0 = false;
          if (more) {
            if (elected) {
#pragma unroll
              for (int k = 0; k < D / 16 - 2; ++k) mma_ss2(tmem + 128, q_lo1 + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
            }
            have_p0 = mbar_test(bar_p_full, (T + 1) & 1);
            if (elected) {
#pragma unroll
              for (int k = D / 16 - 2; k < D / 16; ++k) mma_ss2(tmem + 128, q_lo1 + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
              tc_commit(bar_s_full + 8);
              tc_commit(bar_kv_empty + 8 * kslot);
              if (j + 2 == n) tc_commit(bar_q_empty);
            }
            ok = acquire_kv(j + 1, n);
          }
        }
      }
    }
  } else {
    // ------------------------------------------------- softmax / epilogue warps
    // Warp w works on 16 rows of the current query tile: TMEM lanes 32 (w % 4) + 16 (w / 4) + [0, 16), read in the
    // accumulator-fragment layout (16x256b): thread t holds rows t/4 and t/4 + 8, and of every block of 8
    // columns the two columns 2 (t % 4), 2 (t % 4) + 1.  A row lives in one quad, so its maximum and sum are
    // two shuffles and no warp waits for another.
    const int cq = 2 * (lane & 3);                         // first of this thread's two columns in a block of 8
    // all eight warps work on query tile u = 0, then on tile 1; a warp does 16 rows of each
#define FWD_UNIT(u) const int g = (u), lane_base = (warp & 3) * 32 + (warp >> 2) * 16
    auto quad_max = [](float x) {
      x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
      return fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
    };
    auto quad_sum = [](float x) {
      x += __shfl_xor_sync(0xffffffffu, x, 1);
      return x + __shfl_xor_sync(0xffffffffu, x, 2);
    };
    uint32_t ic = 0, T = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
      const int32_t *I = p.items + (size_t)it * 12;
      const int q_tok0 = I[0], q_pos0 = I[1], q_rows = I[2], head = I[3], a_len = I[5];
      const int b_len = (p.state_mode & STATE_NO_OWN) ? 0 : I[7];
      const int split = (p.state_mode & STATE_OUT) ? 0 : I[8], n_splits = (p.state_mode & STATE_OUT) ? 2 : I[9];
      const int nA = (a_len + 127) >> 7, n = nA + ((b_len + 127) >> 7);
      // per unit u and row (A, B): running reference maximum and this thread's share of the row sum
      float mA[2] = {0.f, 0.f}, mB[2] = {0.f, 0.f}, lA[2] = {0.f, 0.f}, lB[2] = {0.f, 0.f};
      // upper bounds of the rows' scores (log2 units) from the query rows in shared memory and the largest key norm;
      // skip[u]: the warp's rows of unit u have enough headroom to leave the reference maximum where tile 0 put it
      float bndA[2], bndB[2];
      bool skip[2] = {false, false};
      ok = mbar_wait(bar_q_full, ic & 1, ab, WAIT_FWD_Q_FULL);
      if (!ok) break;
      {
        const float kscale = sqrtf(p.kmax2[I[11]]) * p.scale_log2 * 1.0001f;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          FWD_UNIT(u);
          const int rA = lane_base + (lane >> 2), rB = rA + 8;
          float nA2 = 0.f, nB2 = 0.f;
          // a row is NBOX lines of 128 bytes (8 chunks of 16, swizzled among themselves): each thread of the quad
          // squares two chunks of every line, whichever elements they hold
#pragma unroll
          for (int b = 0; b < NBOX; ++b)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              const uint4 xa = *reinterpret_cast<const uint4 *>(smem_raw + SM::kOffQ + g * TILE + b * 16384 + rA * 128 + (((lane & 3) + 4 * c) << 4));
              const uint4 xb = *reinterpret_cast<const uint4 *>(smem_raw + SM::kOffQ + g * TILE + b * 16384 + rB * 128 + (((lane & 3) + 4 * c) << 4));
              const uint32_t wa[4] = {xa.x, xa.y, xa.z, xa.w}, wb[4] = {xb.x, xb.y, xb.z, xb.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&wa[e]));
                const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&wb[e]));
                nA2 = fmaf(fa.x, fa.x, fmaf(fa.y, fa.y, nA2));
                nB2 = fmaf(fb.x, fb.x, fmaf(fb.y, fb.y, nB2));
              }
            }
          bndA[u] = sqrtf(quad_sum(nA2)) * kscale;
          bndB[u] = sqrtf(quad_sum(nB2)) * kscale;
        }
      }
      // the query tiles may be overwritten by the next item's only after every softmax warp has read its rows
      // (this also keeps the softmax warps within one phase of bar_q_full: the next load cannot complete before)
      warp_arrive(bar_q_empty);
      for (int j = 0; j < n && ok; ++j, ++T) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          FWD_UNIT(u);
          const int rA = lane_base + (lane >> 2), rB = rA + 8;   // rows inside the query tile
          const uint32_t lane_off = (uint32_t)lane_base << 16;
          const uint32_t tS = tmem + lane_off + g * 128, tO = tmem + lane_off + 256 + g * 128;
          ok = mbar_wait(bar_s_full + 8 * g, T & 1, ab, WAIT_FWD_S_FULL);
          if (!ok) break;
          tc_fence_after();
          uint32_t s[64];
          tmem_ld_16x256b_x16(tS, s);
          tc_wait_ld();
          // number of leading key columns of this KV tile that rows A and B see
          const int lim0 = (j < nA) ? (a_len - j * 128) : (q_pos0 + g * 128 + 1 - (j - nA) * 128);
          const int limA = (j < nA) ? lim0 : lim0 + rA, limB = (j < nA) ? lim0 : lim0 + rB;
          if (lim0 < 128) {  // same for the whole CTA: a ragged last prompt tile or a tile on the causal diagonal
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const int c = 8 * i + cq;
              if (c >= limA) s[4 * i] = 0xff800000u;       // -inf: exponentiates to zero
              if (c + 1 >= limA) s[4 * i + 1] = 0xff800000u;
              if (c >= limB) s[4 * i + 2] = 0xff800000u;
              if (c + 1 >= limB) s[4 * i + 3] = 0xff800000u;
            }
          }
          if (!skip[u]) {
            // row maxima of the raw scores (the scale is positive, so it commutes with the maximum)
            float xA, xB;
            {
              float a0 = -INFINITY, a1 = -INFINITY, b0 = -INFINITY, b1 = -INFINITY;   // two chains per row: shorter dependency
#pragma unroll
              for (int i = 0; i < 16; i += 2) {
                a0 = max3(a0, __uint_as_float(s[4 * i]), __uint_as_float(s[4 * i + 1]));
                b0 = max3(b0, __uint_as_float(s[4 * i + 2]), __uint_as_float(s[4 * i + 3]));
                a1 = max3(a1, __uint_as_float(s[4 * i + 4]), __uint_as_float(s[4 * i + 5]));
                b1 = max3(b1, __uint_as_float(s[4 * i + 6]), __uint_as_float(s[4 * i + 7]));
              }
              xA = fmaxf(a0, a1);
              xB = fmaxf(b0, b1);
            }
            xA = quad_max(xA) * p.scale_log2;
            xB = quad_max(xB) * p.scale_log2;
            if (j == 0) {
              mA[u] = (xA == -INFINITY) ? 0.f : xA;
              mB[u] = (xB == -INFINITY) ? 0.f : xB;
              skip[u] = __all_sync(0xffffffffu, bndA[u] - mA[u] < kSkipMaxHeadroom && bndB[u] - mB[u] < kSkipMaxHeadroom);
            } else {
              const bool needA = xA > mA[u] + kRescaleThreshold, needB = xB > mB[u] + kRescaleThreshold;
              if (__any_sync(0xffffffffu, needA || needB)) {
                ok = mbar_wait(bar_o_full + 8 * g, (T - 1) & 1, ab, WAIT_FWD_O_FULL);  // PV_g(j-1) done
                if (!ok) break;
                tc_fence_after();
                float alA = 1.f, alB = 1.f;
                if (needA) { alA = ex2(mA[u] - xA); mA[u] = xA; lA[u] *= alA; }
                if (needB) { alB = ex2(mB[u] - xB); mB[u] = xB; lB[u] *= alB; }
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                  uint32_t o[16];
                  tmem_ld_16x256b_x4(tO + c * 32, o);
                  tc_wait_ld();
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    o[4 * i] = __float_as_uint(__uint_as_float(o[4 * i]) * alA);
                    o[4 * i + 1] = __float_as_uint(__uint_as_float(o[4 * i + 1]) * alA);
                    o[4 * i + 2] = __float_as_uint(__uint_as_float(o[4 * i + 2]) * alB);
                    o[4 * i + 3] = __float_as_uint(__uint_as_float(o[4 * i + 3]) * alB);
                  }
                  tmem_st_16x256b_x4(tO + c * 32, o);
                }
              }
            }
          }
          // P = exp2(s * scale - m), bf16 pairs in the 16x128b layout over the S columns [0, 64).  The scale-and-
          // subtract, the row sums and the polynomial exponentials run on register pairs (packed fp32: half the
          // issue slots); kFwdFmaMask says which of the 16 column blocks take their exponentials on the FMA
          // pipe instead of the special-function unit.
          const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
          const float2 nmA = make_float2(-mA[u], -mA[u]), nmB = make_float2(-mB[u], -mB[u]);
          float2 accA = make_float2(0.f, 0.f), accB = make_float2(0.f, 0.f);
          uint32_t pk[32];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float2 xa = __ffma2_rn(make_float2(__uint_as_float(s[4 * i]), __uint_as_float(s[4 * i + 1])), sc2, nmA);
            const float2 xb = __ffma2_rn(make_float2(__uint_as_float(s[4 * i + 2]), __uint_as_float(s[4 * i + 3])), sc2, nmB);
            float2 pa, pb;
            if ((kFwdFmaMask >> i) & 1) { pa = ex2_fma2(xa); pb = ex2_fma2(xb); }
            else { pa = ex2_2(xa); pb = ex2_2(xb); }
            accA = __fadd2_rn(accA, pa);
            accB = __fadd2_rn(accB, pb);
            pk[2 * i] = pack_bf16(pa.x, pa.y);
            pk[2 * i + 1] = pack_bf16(pb.x, pb.y);
          }
          const float sA = accA.x + accA.y, sB = accB.x + accB.y;
          tmem_st_16x128b_x16(tS, pk);
          lA[u] += sA;
          lB[u] += sB;
          tc_wait_st();
          tc_fence_before();
          warp_arrive(bar_p_full + 8 * g);
        }
      }
      if (!ok) break;
      // ---- epilogue: O / l, LSE = ln2 * (m + log2 l); a thread writes two columns of each block of 8 of its rows
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        FWD_UNIT(u);
        const int rA = lane_base + (lane >> 2), rB = rA + 8;
        const uint32_t tO = tmem + ((uint32_t)lane_base << 16) + 256 + g * 128;
        const float ltA = quad_sum(lA[u]), ltB = quad_sum(lB[u]);
        ok = mbar_wait(bar_o_full + 8 * g, (T - 1) & 1, ab, WAIT_FWD_O_FULL);
        if (!ok) break;
        tc_fence_after();
        const float invA = 1.f / ltA, invB = 1.f / ltB;
        const long long tokA = (long long)q_tok0 + g * 128 + rA, tokB = tokA + 8;
        const bool validA = g * 128 + rA < q_rows, validB = g * 128 + rB < q_rows;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[16];
          tmem_ld_16x256b_x4(tO + c * 32, o);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int col = c * 32 + 8 * i + cq;
            if (col >= p.d) continue;  // padding columns of a head dimension below D
            if (n_splits == 1) {
              if (validA) *reinterpret_cast<uint32_t *>(p.o + (tokA * p.h_q + head) * p.d + col) =
                  pack_bf16(__uint_as_float(o[4 * i]) * invA, __uint_as_float(o[4 * i + 1]) * invA);
              if (validB) *reinterpret_cast<uint32_t *>(p.o + (tokB * p.h_q + head) * p.d + col) =
                  pack_bf16(__uint_as_float(o[4 * i + 2]) * invB, __uint_as_float(o[4 * i + 3]) * invB);
            } else {
              if (validA) *reinterpret_cast<float2 *>(p.part_o + (((long long)split * p.n_tok + tokA) * p.h_q + head) * p.d + col) =
                  make_float2(__uint_as_float(o[4 * i]) * invA, __uint_as_float(o[4 * i + 1]) * invA);
              if (validB) *reinterpret_cast<float2 *>(p.part_o + (((long long)split * p.n_tok + tokB) * p.h_q + head) * p.d + col) =
                  make_float2(__uint_as_float(o[4 * i + 2]) * invB, __uint_as_float(o[4 * i + 3]) * invB);
            }
          }
        }
        if ((lane & 3) == 0) {
          const float lseA = (mA[u] + log2f(ltA)) * 0.6931471805599453f, lseB = (mB[u] + log2f(ltB)) * 0.6931471805599453f;
          if (n_splits == 1) {
            if (validA) p.lse[(long long)head * p.n_tok + tokA] = lseA;
            if (validB) p.lse[(long long)head * p.n_tok + tokB] = lseB;
          } else {
            if (validA) p.part_lse[((long long)split * p.h_q + head) * p.n_tok + tokA] = lseA;
            if (validB) p.part_lse[((long long)split * p.h_q + head) * p.n_tok + tokB] = lseB;
          }
        }
        tc_fence_before();
        warp_arrive(bar_o_empty + 8 * g);
      }
      if (ok && warp == 0 && lane == 0) atomicAdd(p.status + 2 + p.kind, 1);  // item finished (work accounting)
    }
  }

  // ---------------------------------------------------------------- teardown
  __syncwarp();
  if (*abort_flag) {
    // give loads that may still be in flight time to land before the CTA's
    // shared memory is released (bounded)
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) {}
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// Merge of up to kMaxStates partial states that live in separate buffers (one per KV shard owner: the states a
// query's owner receives in MoveQ, Sec. 3.3): one warp per (token, head);
// LSE = log sum_s exp(lse_s), O = sum_s exp(lse_s - LSE) O_s.  A shard that saw no key has lse = -inf and weight 0.
constexpr int kMaxStates = 16;
struct StatePtrs {
  const float *o[kMaxStates];    // [tokens, h_q, D] fp32, normalised
  const float *lse[kMaxStates];  // [h_q, tokens]
  int n;
};
template <int D>
__global__ void merge_states_kernel(const StatePtrs sp, __nv_bfloat16 *o, float *lse, long long n_tok, int h_q, int d) {
  const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= n_tok * h_q) return;
  const long long tok = w / h_q;
  const int head = (int)(w % h_q);
  float mx = -INFINITY;
  for (int s = 0; s < sp.n; ++s) mx = fmaxf(mx, sp.lse[s][(long long)head * n_tok + tok]);
  const float ref = mx == -INFINITY ? 0.f : mx;
  float den = 0.f;
  for (int s = 0; s < sp.n; ++s) den += __expf(sp.lse[s][(long long)head * n_tok + tok] - ref);
  constexpr int PER = D / 32;
  float acc[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) acc[i] = 0.f;
  for (int s = 0; s < sp.n; ++s) {
    const float wgt = __expf(sp.lse[s][(long long)head * n_tok + tok] - ref) / den;
    const float *src = sp.o[s] + (tok * h_q + head) * d + lane * PER;
    if (wgt > 0.f && lane * PER < d) {   // (d is a multiple of 8, PER of 2 or 4: a lane is inside or outside as a whole)
#pragma unroll
      for (int i = 0; i < PER; ++i) acc[i] += wgt * src[i];
    }
  }
  __nv_bfloat16 *dst = o + (tok * h_q + head) * d + lane * PER;
  if (lane * PER < d) {
#pragma unroll
    for (int i = 0; i < PER; ++i) dst[i] = __float2bfloat16(acc[i]);
  }
  if (lane == 0) lse[(long long)head * n_tok + tok] = ref + __logf(den);
}

// Largest squared key norm per KV head over the K tensors of one forward call (the unmasked-range tensor and,
// if different, the causal-range tensor): out[h] = max over tokens of |k[token, h, :]|^2, as the bits of a
// non-negative float (so an unsigned atomicMax orders them).  With more than one block per head `out` is cleared by
// the caller before the launch; a single block per head (small inputs) stores its result and needs no clearing.
// Feeds the score bound that lets the tile kernel skip row maxima; HBM-bound, a few microseconds.
template <int D>
__global__ void key_norm_kernel(const __nv_bfloat16 *ka, long long a_tok, const __nv_bfloat16 *kb, long long b_tok, int h_kv,
                                int d, unsigned int *out) {
  constexpr int LPR = D / 8, RPP = 32 / LPR;   // 16-byte loads: lanes per (token, head) row, rows per warp pass
  const int lane = threadIdx.x & 31, sub = lane / LPR, part = lane % LPR;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int head = blockIdx.y;
  float best = 0.f;
  for (int which = 0; which < 2; ++which) {
    const __nv_bfloat16 *k = which ? kb : ka;
    const long long n = which ? b_tok : a_tok;
    for (long long t0 = warp * RPP; t0 < n; t0 += n_warps * RPP) {
      const long long t = t0 + sub;
      float acc = 0.f;
      if (t < n && part * 8 < d) {
        const uint4 x = *reinterpret_cast<const uint4 *>(k + (t * h_kv + head) * d + part * 8);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w[e]));
          acc = fmaf(f.x, f.x, fmaf(f.y, f.y, acc));
        }
      }
#pragma unroll
      for (int sft = LPR / 2; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
      best = fmaxf(best, acc);
    }
  }
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, sft));
  __shared__ float warp_best[32];
  if (lane == 0) warp_best[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < (int)(blockDim.x >> 5); ++i) best = fmaxf(best, warp_best[i]);
    if (gridDim.x == 1) out[head] = __float_as_uint(best);
    else atomicMax(out + head, __float_as_uint(best));
  }
}

// Merge of the prompt-KV shards' partial states (Sec. 3.3): one warp per
// (token, head); LSE = log sum_s exp(lse_s), O = sum_s exp(lse_s - LSE) O_s.
template <int D>
__global__ void combine_kernel(const float *part_o, const float *part_lse, const int32_t *cu_r, const int32_t *branch_group,
                               const int32_t *group_splits, int n_branches, __nv_bfloat16 *o, float *lse,
                               long long n_tok, int h_q, int d) {
  const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= n_tok * h_q) return;
  const long long tok = w / h_q;
  const int head = (int)(w % h_q);
  int lo = 0, hi = n_branches;  // branch b with cu_r[b] <= tok < cu_r[b+1]
  while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cu_r[mid] <= tok) lo = mid; else hi = mid; }
  const int ns = group_splits[branch_group[lo]];
  if (ns == 1) return;  // written directly by the tile kernel
  float mx = -INFINITY;
  for (int s = 0; s < ns; ++s) mx = fmaxf(mx, part_lse[((long long)s * h_q + head) * n_tok + tok]);
  float den = 0.f;
  for (int s = 0; s < ns; ++s) den += __expf(part_lse[((long long)s * h_q + head) * n_tok + tok] - mx);
  constexpr int PER = D / 32;
  float acc[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) acc[i] = 0.f;
  for (int s = 0; s < ns; ++s) {
    const float wgt = __expf(part_lse[((long long)s * h_q + head) * n_tok + tok] - mx) / den;
    const float *src = part_o + (((long long)s * n_tok + tok) * h_q + head) * d + lane * PER;
    if (lane * PER < d) {
#pragma unroll
      for (int i = 0; i < PER; ++i) acc[i] += wgt * src[i];
    }
  }
  __nv_bfloat16 *dst = o + (tok * h_q + head) * d + lane * PER;
  if (lane * PER < d) {
#pragma unroll
    for (int i = 0; i < PER; ++i) dst[i] = __float2bfloat16(acc[i]);
  }
  if (lane == 0) lse[(long long)head * n_tok + tok] = mx + __logf(den);
}

}  // namespace augtree
