// Forward tile kernel: one persistent CTA per replay lane walks its list of
// (pair of query tiles, head) items.  An item's keys are an unmasked range of the
// shared prompt KV followed by a causal range of the query's own sequence
// (Eq. 1); the online-softmax state (m, l, O_acc) of Sec. 3.3 is carried across
// all of the item's KV tiles, which merges the two parts' partial states as it
// goes.  The two query tiles of an item share every K/V tile the CTA loads, and
// each has its own softmax warpgroup, so that one tile's exponentials overlap
// the other tile's MMAs.
//
// Warp roles (320 threads): warps 0-3 own the rows of query tile 0, warps 4-7 the
// rows of query tile 1 (a thread per row: softmax, O rescale, epilogue); warp 8
// lane 0 issues TMA loads; warp 9 lane 0 issues tcgen05 MMAs.
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
  float scale_log2;         // softmax scale * log2(e)
  int *status;
};

constexpr int kFwdThreads = 320;
constexpr float kRescaleThreshold = 8.0f;  // log2 units: P stays <= 2^8

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
    mbar_init(bar_q_full, 1); mbar_init(bar_q_empty, 1);
    for (int s = 0; s < NS; ++s) { mbar_init(bar_kv_full + 8 * s, 1); mbar_init(bar_kv_empty + 8 * s, 1); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(bar_s_full + 8 * g, 1); mbar_init(bar_p_full + 8 * g, 4);
      mbar_init(bar_o_full + 8 * g, 1); mbar_init(bar_o_empty + 8 * g, 4);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 9) { tmem_alloc(smem_u32((const void *)tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const AbortCtx ab{abort_flag, p.status};
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
        const int q_tok0 = I[0], head = I[3], a_tok0 = I[4], a_len = I[5], b_tok0 = I[6], b_len = I[7], kvh = I[11];
        const int nA = (a_len + 127) >> 7, n = nA + ((b_len + 127) >> 7);
        ok = mbar_wait(bar_q_empty, (ic & 1) ^ 1, ab, WAIT_FWD_Q_EMPTY);
        if (!ok) break;
        mbar_expect_tx(bar_q_full, 2 * TILE);
        for (int g = 0; g < 2; ++g)
          for (int b = 0; b < NBOX; ++b) tma_load_3d(sQ + g * TILE + b * 16384, &tm_q, bar_q_full, b * 64, head, q_tok0 + g * 128);
        auto load_tile = [&](bool is_v, int j) -> bool {
          const uint32_t slot = kvc % NS, par = ((kvc / NS) & 1) ^ 1;
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
    if (lane == 0) {
      constexpr uint32_t IDESC_S = make_idesc(128, 128, 0, 0);
      constexpr uint32_t IDESC_PV = make_idesc(128, D, 0, 1);
      uint32_t kvc = 0, ic = 0, T = 0;
      bool ok = true;
      const uint32_t q_lo[2] = {sdesc_lo(sQ, 16), sdesc_lo(sQ + TILE, 16)};
      for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
        const int32_t *I = p.items + (size_t)it * 12;
        const int n = ((I[5] + 127) >> 7) + ((I[7] + 127) >> 7);
        ok = mbar_wait(bar_q_full, ic & 1, ab, WAIT_FWD_Q_FULL);
        if (!ok) break;
        // S_g = Q_g K^T for both query tiles against the K tile in `slot`
        auto issue_s = [&](uint32_t slot) {
          const uint32_t k_lo = sdesc_lo(sKV + slot * TILE, 16);
#pragma unroll
          for (int g = 0; g < 2; ++g) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) mma_ss2(tmem + g * 128, q_lo[g] + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
            tc_commit(bar_s_full + 8 * g);
          }
        };
        {  // prologue: S0(0), S1(0)
          const uint32_t slot = kvc % NS;
          ok = mbar_wait(bar_kv_full + 8 * slot, (kvc / NS) & 1, ab, WAIT_FWD_KV_FULL);
          if (!ok) break;
          tc_fence_after();
          issue_s(slot);
          tc_commit(bar_kv_empty + 8 * slot);
          ++kvc;
          if (n == 1) tc_commit(bar_q_empty);
        }
        for (int j = 0; j < n && ok; ++j, ++T) {
          const uint32_t vslot = kvc % NS;
          ok = mbar_wait(bar_kv_full + 8 * vslot, (kvc / NS) & 1, ab, WAIT_FWD_KV_FULL);
          if (!ok) break;
          ++kvc;
          uint32_t kslot = 0;
          const bool more = j + 1 < n;
          if (more) {
            kslot = kvc % NS;
            ok = mbar_wait(bar_kv_full + 8 * kslot, (kvc / NS) & 1, ab, WAIT_FWD_KV_FULL);
            if (!ok) break;
            ++kvc;
          }
          const uint32_t v_lo = sdesc_lo(sKV + vslot * TILE, 16384);
          const uint32_t k_lo = sdesc_lo(sKV + kslot * TILE, 16);
          const uint32_t acc0 = j > 0 ? 1u : 0u;
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            // PV_g(j): P_g (bf16, over S_g) times V
            ok = mbar_wait(bar_p_full + 8 * g, T & 1, ab, WAIT_FWD_P_FULL);
            if (!ok) break;
            if (j == 0 && ic > 0) {
              ok = mbar_wait(bar_o_empty + 8 * g, (ic - 1) & 1, ab, WAIT_FWD_O_EMPTY);
              if (!ok) break;
            }
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < 8; ++k)
              mma_ts2(tmem + 256 + g * 128, tmem + g * 128 + k * 8, v_lo + kstep_mnmajor(k), IDESC_PV, acc0 | (uint32_t)(k > 0));
            tc_commit(bar_o_full + 8 * g);
            if (g == 1) tc_commit(bar_kv_empty + 8 * vslot);
            // S_g(j+1) overwrites P_g(j): the tensor pipe runs in order
            if (more) {
#pragma unroll
              for (int k = 0; k < D / 16; ++k) mma_ss2(tmem + g * 128, q_lo[g] + kstep_kmajor(k), k_lo + kstep_kmajor(k), IDESC_S, k > 0);
              tc_commit(bar_s_full + 8 * g);
              if (g == 1) {
                tc_commit(bar_kv_empty + 8 * kslot);
                if (j + 2 == n) tc_commit(bar_q_empty);
              }
            }
          }
        }
      }
    }
  } else {
    // ------------------------------------------------- softmax / epilogue warps
    const int g = warp >> 2;                 // query tile of the pair
    const int r = (warp & 3) * 32 + lane;    // row inside the tile == TMEM lane
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_off + g * 128, tO = tmem + lane_off + 256 + g * 128;
    uint32_t ic = 0, T = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
      const int32_t *I = p.items + (size_t)it * 12;
      const int q_tok0 = I[0], q_pos0 = I[1], q_rows = I[2], head = I[3], a_len = I[5], b_len = I[7];
      const int split = I[8], n_splits = I[9];
      const int nA = (a_len + 127) >> 7, n = nA + ((b_len + 127) >> 7);
      const int my_pos = q_pos0 + g * 128 + r;  // position of this row in its sequence
      float m_used = 0.f, l = 0.f;
      for (int j = 0; j < n; ++j, ++T) {
        ok = mbar_wait(bar_s_full + 8 * g, T & 1, ab, WAIT_FWD_S_FULL);
        if (!ok) break;
        tc_fence_after();
        // number of leading key columns of this tile that the row sees
        const int limit = (j < nA) ? (a_len - j * 128) : (my_pos + 1 - (j - nA) * 128);
        // pass 1: row maximum of the raw scores (the scale is positive, so it commutes with the maximum);
        // 64 columns per TMEM round trip
        float mx = -INFINITY;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t sv[64];
          tmem_ld32(tS + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
          tmem_ld32(tS + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
          tc_wait_ld();
          if (limit >= 128) {
#pragma unroll
            for (int i = 0; i < 64; ++i) mx = fmaxf(mx, __uint_as_float(sv[i]));
          } else {
#pragma unroll
            for (int i = 0; i < 64; ++i)
              if (h * 64 + i < limit) mx = fmaxf(mx, __uint_as_float(sv[i]));
          }
        }
        mx *= p.scale_log2;
        if (j == 0) {
          m_used = (mx == -INFINITY) ? 0.f : mx;
        } else {
          const bool need = mx > m_used + kRescaleThreshold;
          if (__any_sync(0xffffffffu, need)) {
            ok = mbar_wait(bar_o_full + 8 * g, (T - 1) & 1, ab, WAIT_FWD_O_FULL);  // PV_g(j-1) done
            if (!ok) break;
            tc_fence_after();
            float alpha = 1.f;
            if (need) { alpha = ex2(m_used - mx); m_used = mx; l *= alpha; }
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(tO + c * 32, o);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              tmem_st32(tO + c * 32, o);
            }
          }
        }
        // pass 2: P = exp2(s * scale - m) from a second read of S; P (bf16) overwrites S columns
        // [16c, 16c+16), which lie inside the columns [0, 32c+32) this thread has already consumed
        float sum = 0.f;
        uint32_t sa[32], sb[32];  // the next 32 columns are in flight while the current ones are exponentiated
        tmem_ld32(tS, sa);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t (&cur)[32] = (c & 1) ? sb : sa;
          uint32_t (&nxt)[32] = (c & 1) ? sa : sb;
          tc_wait_ld();
          if (c < 3) tmem_ld32(tS + (c + 1) * 32, nxt);
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float p0 = ex2(fmaf(__uint_as_float(cur[2 * i]), p.scale_log2, -m_used));
            float p1 = ex2(fmaf(__uint_as_float(cur[2 * i + 1]), p.scale_log2, -m_used));
            if (limit < 128) {
              if (c * 32 + 2 * i >= limit) p0 = 0.f;
              if (c * 32 + 2 * i + 1 >= limit) p1 = 0.f;
            }
            sum += p0 + p1;
            pk[i] = pack_bf16(p0, p1);
          }
          tmem_st16(tS + c * 16, pk);
        }
        l += sum;
        tc_wait_st();
        tc_fence_before();
        warp_arrive(bar_p_full + 8 * g);
      }
      if (!ok) break;
      // ---- epilogue: O / l, LSE = ln2 * (m + log2 l)
      ok = mbar_wait(bar_o_full + 8 * g, (T - 1) & 1, ab, WAIT_FWD_O_FULL);
      if (!ok) break;
      tc_fence_after();
      const float inv_l = 1.f / l;
      const long long tok = (long long)q_tok0 + g * 128 + r;
      const bool valid = g * 128 + r < q_rows;
      const float lse = (m_used + log2f(l)) * 0.6931471805599453f;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(tO + c * 32, o);
        tc_wait_ld();
        if (valid) {
          if (n_splits == 1) {
            uint4 *dst = reinterpret_cast<uint4 *>(p.o + (tok * p.h_q + head) * D + c * 32);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint4 w;
              w.x = pack_bf16(__uint_as_float(o[8 * v + 0]) * inv_l, __uint_as_float(o[8 * v + 1]) * inv_l);
              w.y = pack_bf16(__uint_as_float(o[8 * v + 2]) * inv_l, __uint_as_float(o[8 * v + 3]) * inv_l);
              w.z = pack_bf16(__uint_as_float(o[8 * v + 4]) * inv_l, __uint_as_float(o[8 * v + 5]) * inv_l);
              w.w = pack_bf16(__uint_as_float(o[8 * v + 6]) * inv_l, __uint_as_float(o[8 * v + 7]) * inv_l);
              dst[v] = w;
            }
          } else {
            float4 *dst = reinterpret_cast<float4 *>(p.part_o + (((long long)split * p.n_tok + tok) * p.h_q + head) * D + c * 32);
#pragma unroll
            for (int v = 0; v < 8; ++v)
              dst[v] = make_float4(__uint_as_float(o[4 * v]) * inv_l, __uint_as_float(o[4 * v + 1]) * inv_l,
                                   __uint_as_float(o[4 * v + 2]) * inv_l, __uint_as_float(o[4 * v + 3]) * inv_l);
          }
        }
      }
      if (valid) {
        if (n_splits == 1) p.lse[(long long)head * p.n_tok + tok] = lse;
        else p.part_lse[((long long)split * p.h_q + head) * p.n_tok + tok] = lse;
      }
      tc_fence_before();
      warp_arrive(bar_o_empty + 8 * g);
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

// Merge of the prompt-KV shards' partial states (Sec. 3.3): one warp per
// (token, head); LSE = log sum_s exp(lse_s), O = sum_s exp(lse_s - LSE) O_s.
template <int D>
__global__ void combine_kernel(const float *part_o, const float *part_lse, const int32_t *cu_r, const int32_t *branch_group,
                               const int32_t *group_splits, int n_branches, __nv_bfloat16 *o, float *lse,
                               long long n_tok, int h_q) {
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
    const float *src = part_o + (((long long)s * n_tok + tok) * h_q + head) * D + lane * PER;
#pragma unroll
    for (int i = 0; i < PER; ++i) acc[i] += wgt * src[i];
  }
  __nv_bfloat16 *dst = o + (tok * h_q + head) * D + lane * PER;
#pragma unroll
  for (int i = 0; i < PER; ++i) dst[i] = __float2bfloat16(acc[i]);
  if (lane == 0) lse[(long long)head * n_tok + tok] = mx + __logf(den);
}

}  // namespace augtree
