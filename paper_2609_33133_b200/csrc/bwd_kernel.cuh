// Backward tile kernel, KV-stationary: one persistent CTA per replay lane walks
// its list of (KV tile, KV head) items.  An item keeps its K and V tile in
// shared memory and streams past it every query tile that can see it: for a
// prompt-KV tile in replay, all response tiles of all G branches and all
// query heads of the KV head, which is the many-to-one sum of Eq. 2 done in
// one TMEM accumulator in a fixed order; for a tile inside a sequence, the
// causal query tiles of that sequence.
//
// Per (KV tile, Q tile, head) pair, with S^T = K Q^T so that a thread owns a key:
//   P^T = exp2(S^T * scale*log2e - lse2[q]),  dP^T = V dO^T,
//   dS^T = scale * P^T * (dP^T - delta[q]),
//   dV += P^T dO,  dK += dS^T Q,  dQ[q,:] += dS K   (dQ leaves through fp32 atomics).
//
// Warp roles (192 threads): warps 0-3 element-wise work and epilogues, warp 4
// lane 0 TMA, warp 5 lane 0 MMA.  TMEM columns: T0 [0,128) holds S^T, then P^T
// (bf16, columns 0-63) and the low half of dQ (columns 64-127); T1 [128,256)
// holds dP^T, then dS^T and the high half of dQ; dV at 256, dK at 256 + D.
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace augtree {

struct BwdParams {
  const int32_t *items;     // lane order, 8 ints each
  const int32_t *lane_ptr;  // [gridDim.x + 1]
  const int32_t *segs;      // [n_seg][2] {first query token, length}
  const float *lse2;        // [h_q, n_tok]  lse * log2(e)
  const float *delta;       // [h_q, n_tok]  rowsum(dO * O)
  float *dq_acc;            // [n_tok, h_q, D] fp32, zeroed by the caller
  __nv_bfloat16 *dk_out, *dv_out;  // mode-0 items when causal_fp32 == 0: [kv tokens, h_kv, D] bf16
  float *dk_acc, *dv_acc;   // fp32 [prompt tokens, h_kv, D]: mode-1 items, and mode-0 items when causal_fp32 != 0
  long long n_tok;          // tokens of the query tensor
  int h_q, h_kv;
  int causal_fp32;
  float scale, scale_log2;
  int *status;
};

constexpr int kBwdThreads = 192;
constexpr int kBwdStages = 2;

template <int D>
struct BwdSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kDsBytes = 128 * 128 * 2;
  static constexpr int kOffK = 0, kOffV = kTileBytes, kOffQ = 2 * kTileBytes;  // Q[s], dO[s] interleaved per stage
  static constexpr int kOffDs = kOffQ + 2 * kBwdStages * kTileBytes;
  static constexpr int kOffRow = kOffDs + kDsBytes;  // lse2[128], delta[128] of the current query tile
  static constexpr int kOffBar = kOffRow + 2 * 128 * 4;
  static constexpr int kBytes = kOffBar + 160 + 1024;
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
           const __grid_constant__ CUtensorMap tm_k0, const __grid_constant__ CUtensorMap tm_v0,
           const __grid_constant__ CUtensorMap tm_k1, const __grid_constant__ CUtensorMap tm_v1, const BwdParams p) {
  using SM = BwdSmem<D>;
  constexpr int TILE = SM::kTileBytes;
  constexpr int NBOX = D / 64;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sK = base + SM::kOffK, sV = base + SM::kOffV, sQ0 = base + SM::kOffQ, sDs = base + SM::kOffDs;
  float *rb = reinterpret_cast<float *>(gen + SM::kOffRow);  // [2][128]
  const uint32_t bars = base + SM::kOffBar;
  const uint32_t bar_kv_full = bars, bar_kv_empty = bars + 8;
  const uint32_t bar_qdo_full = bars + 16, bar_qdo_empty = bars + 32;  // [2] each
  const uint32_t bar_s_full = bars + 48, bar_pds_full = bars + 56, bar_mma2 = bars + 64, bar_dq_free = bars + 72;
  const uint32_t bar_acc_full = bars + 80, bar_acc_empty = bars + 88, bar_rows = bars + 96;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen + SM::kOffBar + 104);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(gen + SM::kOffBar + 112);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar_kv_full, 1); mbar_init(bar_kv_empty, 1);
    for (int s = 0; s < kBwdStages; ++s) { mbar_init(bar_qdo_full + 8 * s, 1); mbar_init(bar_qdo_empty + 8 * s, 1); }
    mbar_init(bar_s_full, 1); mbar_init(bar_pds_full, 128); mbar_init(bar_mma2, 1); mbar_init(bar_dq_free, 128);
    mbar_init(bar_acc_full, 1); mbar_init(bar_acc_empty, 128); mbar_init(bar_rows, 128);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 5) { tmem_alloc(smem_u32((const void *)tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tT0 = tmem, tT1 = tmem + 128, tDV = tmem + 256, tDK = tmem + 256 + D;
  const AbortCtx ab{abort_flag, p.status};
  const int rep = p.h_q / p.h_kv;
  const int it_begin = p.lane_ptr[blockIdx.x], it_end = p.lane_ptr[blockIdx.x + 1];

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_do); tma_prefetch_desc(&tm_k0);
      tma_prefetch_desc(&tm_v0); tma_prefetch_desc(&tm_k1); tma_prefetch_desc(&tm_v1);
      uint32_t ic = 0, T = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
        const int32_t *I = p.items + (size_t)it * 8;
        const int kv_tok0 = I[0], kv_pos0 = I[1], kvh = I[3], mode = I[4], seg0 = I[5], nseg = I[6];
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
          const int s_tok0 = p.segs[2 * sg], s_len = p.segs[2 * sg + 1];
          const int nqt = (s_len + 127) >> 7;
          for (int qt = mode ? 0 : (kv_pos0 >> 7); qt < nqt && ok; ++qt)
            for (int j = 0; j < rep; ++j, ++T) {
              const uint32_t st = T % kBwdStages, par = ((T / kBwdStages) & 1) ^ 1;
              ok = mbar_wait(bar_qdo_empty + 8 * st, par, ab, WAIT_BWD_QDO_EMPTY);
              if (!ok) break;
              mbar_expect_tx(bar_qdo_full + 8 * st, 2 * TILE);
              const uint32_t dq = sQ0 + st * 2 * TILE, ddo = dq + TILE;
              for (int b = 0; b < NBOX; ++b) {
                tma_load_3d(dq + b * 16384, &tm_q, bar_qdo_full + 8 * st, b * 64, kvh * rep + j, s_tok0 + qt * 128);
                tma_load_3d(ddo + b * 16384, &tm_do, bar_qdo_full + 8 * st, b * 64, kvh * rep + j, s_tok0 + qt * 128);
              }
            }
        }
      }
    }
  } else if (warp == 5) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC_ST = make_idesc(128, 128, 0, 0);  // S^T, dP^T: both operands K-major
      constexpr uint32_t IDESC_ACC = make_idesc(128, D, 0, 1);   // dV, dK: A from TMEM, B = dO / Q MN-major
      constexpr uint32_t IDESC_DQ = make_idesc(128, 64, 1, 1);   // dQ halves: A = dS MN-major, B = K MN-major
      uint32_t ic = 0, T = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
        const int32_t *I = p.items + (size_t)it * 8;
        const int kv_pos0 = I[1], mode = I[4], seg0 = I[5], nseg = I[6];
        ok = mbar_wait(bar_kv_full, ic & 1, ab, WAIT_BWD_KV_FULL);
        if (!ok) break;
        bool first = true;
        for (int sg = seg0; sg < seg0 + nseg && ok; ++sg) {
          const int nqt = (p.segs[2 * sg + 1] + 127) >> 7;
          for (int qt = mode ? 0 : (kv_pos0 >> 7); qt < nqt && ok; ++qt)
            for (int j = 0; j < rep; ++j, ++T) {
              const uint32_t st = T % kBwdStages;
              const uint32_t sQ = sQ0 + st * 2 * TILE, sdO = sQ + TILE;
              ok = mbar_wait(bar_qdo_full + 8 * st, (T / kBwdStages) & 1, ab, WAIT_BWD_QDO_FULL);
              if (!ok) break;
              if (T > 0) {
                ok = mbar_wait(bar_dq_free, (T - 1) & 1, ab, WAIT_BWD_DQ_FREE);
                if (!ok) break;
              }
              tc_fence_after();
#pragma unroll
              for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = (k >> 2) * 16384 + (k & 3) * 32;
                mma_ss(tT0, make_sdesc(sK + off, 16, 1024), make_sdesc(sQ + off, 16, 1024), IDESC_ST, k > 0);
              }
#pragma unroll
              for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = (k >> 2) * 16384 + (k & 3) * 32;
                mma_ss(tT1, make_sdesc(sV + off, 16, 1024), make_sdesc(sdO + off, 16, 1024), IDESC_ST, k > 0);
              }
              tc_commit(bar_s_full);
              ok = mbar_wait(bar_pds_full, T & 1, ab, WAIT_BWD_PDS_FULL);
              if (!ok) break;
              if (first && ic > 0) {
                ok = mbar_wait(bar_acc_empty, (ic - 1) & 1, ab, WAIT_BWD_ACC_EMPTY);
                if (!ok) break;
              }
              tc_fence_after();
              const uint32_t acc0 = first ? 0u : 1u;
#pragma unroll
              for (int k = 0; k < 8; ++k)
                mma_ts(tDV, tT0 + k * 8, make_sdesc(sdO + k * 2048, 16384, 1024), IDESC_ACC, acc0 | (k > 0));
#pragma unroll
              for (int k = 0; k < 8; ++k)
                mma_ts(tDK, tT1 + k * 8, make_sdesc(sQ + k * 2048, 16384, 1024), IDESC_ACC, acc0 | (k > 0));
#pragma unroll
              for (int h = 0; h < NBOX; ++h)
#pragma unroll
                for (int k = 0; k < 8; ++k)
                  mma_ss((h ? tT1 : tT0) + 64, make_sdesc(sDs + k * 2048, 16384, 1024),
                         make_sdesc(sK + h * 16384 + k * 2048, 16384, 1024), IDESC_DQ, k > 0);
              tc_commit(bar_mma2);
              tc_commit(bar_qdo_empty + 8 * st);
              first = false;
            }
        }
        if (!ok) break;
        tc_commit(bar_acc_full);
        tc_commit(bar_kv_empty);
      }
    }
  } else {
    // ------------------------------------------------------- compute warps 0-3
    const int t = threadIdx.x;  // TMEM lane: key row for S^T/dP^T/dV/dK, query row for dQ
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    uint32_t ic = 0, T = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end && ok; ++it, ++ic) {
      const int32_t *I = p.items + (size_t)it * 8;
      const int kv_tok0 = I[0], kv_pos0 = I[1], kv_rows = I[2], kvh = I[3], mode = I[4], seg0 = I[5], nseg = I[6];
      const bool key_valid = t < kv_rows;
      for (int sg = seg0; sg < seg0 + nseg && ok; ++sg) {
        const int s_tok0 = p.segs[2 * sg], s_len = p.segs[2 * sg + 1];
        const int nqt = (s_len + 127) >> 7;
        for (int qt = mode ? 0 : (kv_pos0 >> 7); qt < nqt && ok; ++qt)
          for (int j = 0; j < rep; ++j, ++T) {
            const int head = kvh * rep + j;
            const int q_rows = min(128, s_len - qt * 128);
            const long long tok = (long long)s_tok0 + qt * 128 + t;
            {
              const bool qv = t < q_rows;
              rb[t] = qv ? p.lse2[(long long)head * p.n_tok + tok] : INFINITY;
              rb[128 + t] = qv ? p.delta[(long long)head * p.n_tok + tok] : 0.f;
            }
            mbar_arrive(bar_rows);
            ok = mbar_wait(bar_rows, T & 1, ab, WAIT_BWD_ROWS);
            if (!ok) break;
            ok = mbar_wait(bar_s_full, T & 1, ab, WAIT_BWD_S_FULL);
            if (!ok) break;
            tc_fence_after();
            // first query column this key may NOT be hidden from: col >= lo is visible
            const int lo = mode ? 0 : (kv_pos0 + t - qt * 128);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t sv[32], dpv[32];
              tmem_ld32(tT0 + lane_off + c * 32, sv);
              tmem_ld32(tT1 + lane_off + c * 32, dpv);
              tc_wait_ld();
              uint32_t pp[16], dd[16];
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                float pv[2], dv[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                  const int col = c * 32 + 2 * i + e;
                  const float l2 = rb[col], dl = rb[128 + col];
                  float pr = ex2(__uint_as_float(sv[2 * i + e]) * p.scale_log2 - l2);
                  if (!key_valid || col < lo) pr = 0.f;
                  pv[e] = pr;
                  dv[e] = pr * (__uint_as_float(dpv[2 * i + e]) - dl) * p.scale;
                }
                pp[i] = pack_bf16(pv[0], pv[1]);
                dd[i] = pack_bf16(dv[0], dv[1]);
              }
              tmem_st16(tT0 + lane_off + c * 16, pp);
              tmem_st16(tT1 + lane_off + c * 16, dd);
              // dS^T row t, query columns [32c, 32c+32) -> shared, MN-major (query contiguous), 128B swizzle
              uint8_t *row = gen + SM::kOffDs + (c >> 1) * 16384 + t * 128;
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                const int chunk = (c & 1) * 4 + v;
                *reinterpret_cast<uint4 *>(row + ((chunk ^ (t & 7)) << 4)) =
                    make_uint4(dd[4 * v], dd[4 * v + 1], dd[4 * v + 2], dd[4 * v + 3]);
              }
            }
            tc_wait_st();
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar_pds_full);
            // ---- drain dQ of this pair: thread t owns query row t
            ok = mbar_wait(bar_mma2, T & 1, ab, WAIT_BWD_MMA2);
            if (!ok) break;
            tc_fence_after();
            {
              const bool qv = t < q_rows;
              float *dst = p.dq_acc + (tok * p.h_q + head) * D;
#pragma unroll
              for (int h = 0; h < NBOX; ++h)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                  uint32_t v[32];
                  tmem_ld32((h ? tT1 : tT0) + lane_off + 64 + c * 32, v);
                  tc_wait_ld();
                  if (qv) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                      red_add_v4(dst + h * 64 + c * 32 + 4 * i, __uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                 __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                  }
                }
            }
            tc_fence_before();
            mbar_arrive(bar_dq_free);
          }
      }
      if (!ok) break;
      // ---- item epilogue: dV, dK of key row t
      ok = mbar_wait(bar_acc_full, ic & 1, ab, WAIT_BWD_ACC_FULL);
      if (!ok) break;
      tc_fence_after();
      const long long krow = ((long long)kv_tok0 + t) * p.h_kv + kvh;
      const bool to_fp32 = mode || p.causal_fp32;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t v[32];
          tmem_ld32((which ? tDK : tDV) + lane_off + c * 32, v);
          tc_wait_ld();
          if (key_valid) {
            if (to_fp32) {
              float4 *dst = reinterpret_cast<float4 *>((which ? p.dk_acc : p.dv_acc) + krow * D + c * 32);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                float4 a = dst[i];
                a.x += __uint_as_float(v[4 * i]); a.y += __uint_as_float(v[4 * i + 1]);
                a.z += __uint_as_float(v[4 * i + 2]); a.w += __uint_as_float(v[4 * i + 3]);
                dst[i] = a;
              }
            } else {
              uint4 *dst = reinterpret_cast<uint4 *>((which ? p.dk_out : p.dv_out) + krow * D + c * 32);
#pragma unroll
              for (int i = 0; i < 4; ++i)
                dst[i] = make_uint4(pack_bf16(__uint_as_float(v[8 * i]), __uint_as_float(v[8 * i + 1])),
                                    pack_bf16(__uint_as_float(v[8 * i + 2]), __uint_as_float(v[8 * i + 3])),
                                    pack_bf16(__uint_as_float(v[8 * i + 4]), __uint_as_float(v[8 * i + 5])),
                                    pack_bf16(__uint_as_float(v[8 * i + 6]), __uint_as_float(v[8 * i + 7])));
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar_acc_empty);
    }
  }

  __syncwarp();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) {}
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// delta[h, tok] = sum_d dO * O  and  lse2 = lse * log2(e); one warp per (token, head).
template <int D>
__global__ void bwd_preprocess_kernel(const __nv_bfloat16 *o, const __nv_bfloat16 *d_o, const float *lse, float *delta,
                                      float *lse2, long long n_tok, int h_q) {
  const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= n_tok * h_q) return;
  const long long tok = w / h_q;
  const int head = (int)(w % h_q);
  constexpr int PER = D / 32;
  const __nv_bfloat16 *po = o + w * D + lane * PER, *pd = d_o + w * D + lane * PER;
  float acc = 0.f;
#pragma unroll
  for (int i = 0; i < PER; ++i) acc += __bfloat162float(po[i]) * __bfloat162float(pd[i]);
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (lane == 0) {
    delta[(long long)head * n_tok + tok] = acc;
    lse2[(long long)head * n_tok + tok] = lse[(long long)head * n_tok + tok] * 1.4426950408889634f;
  }
}

// fp32 -> bf16 (dQ accumulator, optional bf16 copies of the prompt gradients)
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
