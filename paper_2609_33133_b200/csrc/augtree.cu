// C-ABI entry points: plan lifetime, tensor-map encoding and kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>

#include "bwd_kernel.cuh"
#include "dq_kernel.cuh"
#include "dql_kernel.cuh"
#include "fwd_kernel.cuh"
#include "plan.h"

using namespace augtree;

// Built-in scratch of augtree_replay_fwd_static: part of the device image, so
// each GPU that loads this library holds it until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[AUGTREE_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxStaticDevices = 64;
void *g_static_ptr[kMaxStaticDevices] = {};  // device address of g_static_scratch, per device
std::mutex g_static_mutex;

std::atomic<long long> g_launches{0};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  });
  return fn;
}

// Tensor map over a packed [tokens, heads, d] bf16 tensor; one box = 128 tokens
// of one head, 64 elements (128 bytes) wide, written to shared memory with the
// 128-byte swizzle.  Rows past the end of the tensor read as zero.
int make_map(CUtensorMap *m, const void *ptr, long long tokens, int heads, int d) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return AUGTREE_ERR_CUDA;
  if (tokens < 1) tokens = 1;
  const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)heads, (cuuint64_t)tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)heads * d * 2};
  const cuuint32_t box[3] = {64, 1, 128};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? AUGTREE_OK : AUGTREE_ERR_CUDA;
}

// Tensor map over the dS hand-off scratch: [slots][128 keys][128 queries] bf16, one box = 64 queries of all 128
// keys of one slot (the MN-major A operand of the query-side GEMM, 128-byte swizzle).
int make_ds_map(CUtensorMap *m, const void *ptr, long long slots) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return AUGTREE_ERR_CUDA;
  if (slots < 1) slots = 1;
  const cuuint64_t dims[3] = {128, 128, (cuuint64_t)slots};
  const cuuint64_t strides[2] = {256, 32768};
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? AUGTREE_OK : AUGTREE_ERR_CUDA;
}

constexpr size_t kFwdHeaderBytes = 256;  // head of the forward scratch: per-KV-head key-norm maxima (plan.cpp reserves it)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
size_t al256(size_t x) { return (x + 255) & ~(size_t)255; }

int upload(const std::vector<int32_t> &h, int32_t **d) {
  *d = nullptr;
  const size_t bytes = (h.size() ? h.size() : 1) * sizeof(int32_t);
  if (cudaMalloc(d, bytes) != cudaSuccess) return AUGTREE_ERR_CUDA;
  if (!h.empty() && cudaMemcpy(*d, h.data(), h.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
    return AUGTREE_ERR_CUDA;
  return AUGTREE_OK;
}

int upload_sched(Sched &s, int n_lanes, bool drop_last) {
  std::vector<int32_t> sorted(s.items.size());
  for (size_t i = 0; i < s.order.size(); ++i)
    std::memcpy(&sorted[i * s.item_ints], &s.items[(size_t)s.order[i] * s.item_ints], s.item_ints * sizeof(int32_t));
  int r = upload(sorted, &s.d_items);
  if (r) return r;
  if (!drop_last) return upload(s.lane_ptr, &s.d_lane_ptr);
  // injected fault (AUGTREE_FLAG_TEST_DROP_ITEM): the device copy of the lane table loses the last item of the
  // last lane that has one; the host tables and the expected item count stay whole
  std::vector<int32_t> lp = s.lane_ptr;
  for (int l = n_lanes; l > 0; --l)
    if (lp[l] > lp[l - 1]) {
      for (int k = l; k <= n_lanes; ++k) --lp[k];
      break;
    }
  return upload(lp, &s.d_lane_ptr);
}

void timing_mark(const augtree_plan *pl, int kind, bool stop, cudaStream_t st);

long long wait_budget(const augtree_plan *pl) {
  return (pl->flags & AUGTREE_FLAG_TEST_SHORT_WAIT) ? kWaitBudgetClocksTest : kWaitBudgetClocks;
}

template <int D>
int launch_fwd(const augtree_plan *pl, const Sched &s, const void *q, long long q_tok, const void *ka, const void *va,
               long long a_tok, const void *kb, const void *vb, long long b_tok, void *o, float *lse, float *part_o,
               float *part_lse, void *ws, cudaStream_t st, int state_mode = 0) {
  if (s.n_items() == 0) return AUGTREE_OK;
  // first 256 bytes of the scratch: largest squared key norm per KV head (score bound of the tile kernel)
  unsigned int *kmax2 = static_cast<unsigned int *>(ws);
  {
    const bool same = ka == kb;
    const long long rows = a_tok + (same ? 0 : b_tok);
    // small inputs: one block per head, which stores its maximum (no clearing launch); otherwise clear, then atomicMax
    const unsigned blocks = rows <= 4096 ? 1u : (unsigned)std::min<long long>(2368, rows / 64);
    if (blocks > 1 && cudaMemsetAsync(kmax2, 0, (size_t)pl->h_kv * sizeof(unsigned int), st) != cudaSuccess) return AUGTREE_ERR_CUDA;
    key_norm_kernel<D><<<dim3(blocks, (unsigned)pl->h_kv), 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(ka), a_tok,
                                                                       static_cast<const __nv_bfloat16 *>(kb), same ? 0 : b_tok,
                                                                       pl->h_kv, pl->head_dim, kmax2);
    ++g_launches;
  }
  CUtensorMap mq, mka, mva, mkb, mvb;
  int r;
  if ((r = make_map(&mq, q, q_tok, pl->h_q, pl->head_dim))) return r;
  if ((r = make_map(&mka, ka, a_tok, pl->h_kv, pl->head_dim))) return r;
  if ((r = make_map(&mva, va, a_tok, pl->h_kv, pl->head_dim))) return r;
  if ((r = make_map(&mkb, kb, b_tok, pl->h_kv, pl->head_dim))) return r;
  if ((r = make_map(&mvb, vb, b_tok, pl->h_kv, pl->head_dim))) return r;
  FwdParams p;
  p.items = s.d_items; p.lane_ptr = s.d_lane_ptr;
  p.o = static_cast<__nv_bfloat16 *>(o); p.lse = lse; p.part_o = part_o; p.part_lse = part_lse;
  p.n_tok = q_tok; p.h_q = pl->h_q; p.d = pl->head_dim; p.scale_log2 = pl->scale * 1.4426950408889634f; p.status = pl->d_status;
  p.kmax2 = reinterpret_cast<const float *>(kmax2);
  const int kind = (int)(&s - pl->sched);
  p.wait_budget = wait_budget(pl); p.kind = kind;
  p.test_flags = (pl->flags & AUGTREE_FLAG_TEST_SKIP_FWD_LOAD) ? TEST_SKIP_FWD_LOAD : 0;
  p.state_mode = state_mode;
  pl->launched_items[kind] += s.n_items();
  timing_mark(pl, kind, false, st);
  fwd_kernel<D><<<pl->n_lanes, kFwdThreads, FwdSmem<D>::kBytes, st>>>(mq, mka, mva, mkb, mvb, p);
  timing_mark(pl, kind, true, st);
  ++g_launches;
  return cudaGetLastError() == cudaSuccess ? AUGTREE_OK : AUGTREE_ERR_CUDA;
}

struct BwdArgs {
  const void *q, *d_o, *o;
  const float *lse;
  long long q_tok;
  const void *k0, *v0; long long kv0_tok;  // mode-0 K/V tensor (the queries' own sequence)
  const void *k1, *v1; long long kv1_tok;  // mode-1 K/V tensor (shared prompt)
  void *dq; void *dk_out, *dv_out;
  float *dk_acc, *dv_acc;
  int causal_fp32;
  const int32_t *d_segs;
  const int32_t *d_tiles;  // [n_tiles][2] query tiles of the call's query tensor
  long long n_tiles;
  const Sched *dq_sched;   // query-side units
  // key ranges of the query-side kernel: unmasked range tensor (a), causal range tensor (b)
  const void *ka, *va; long long a_tok;
  int no_own = 0;           // partial-state variant: only the plan's prompt keys (mode-1 items, no causal range in dQ)
  float *dq_f32 = nullptr;  // partial-state variant: fp32 dQ contribution
  const int32_t *d_pairs = nullptr;  // dS hand-off table of the call's query tiles
  long long ds_slots = 0;            // (KV tile, query tile) pairs per head of the call
};

// One backward call: row statistics, then the key-side kernel (dK, dV), then the query-side kernel (dQ).
// With scratch for it (ws_bytes >= the plan's hand-off size) the key-side kernel also stores dS and the
// query side is one GEMM per pair (dql_kernel); otherwise the query side recomputes S and dP (dq_kernel).
template <int D>
int launch_bwd(const augtree_plan *pl, const Sched &s, const BwdArgs &a, void *ws, size_t ws_bytes, cudaStream_t st) {
  if (a.q_tok == 0) return AUGTREE_OK;
  float *stats = static_cast<float *>(ws);
  // (the hand-off tiles are written with 32-byte stores: the scratch must be aligned to that, else the recomputing path)
  const bool handoff = ws_bytes >= pl->ws_bwd_handoff && s.n_items() > 0 && a.dq_sched->n_items() > 0 &&
                       (reinterpret_cast<uintptr_t>(ws) & 31u) == 0;
  __nv_bfloat16 *ds = handoff ? reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(ws) + pl->ws_bwd) : nullptr;
  {
    const dim3 grid((unsigned)a.n_tiles, (unsigned)pl->h_q);
    bwd_preprocess_kernel<D><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(a.o), static_cast<const __nv_bfloat16 *>(a.d_o),
                                                   a.lse, a.d_tiles, stats, a.q_tok, a.n_tiles, pl->h_q, pl->head_dim, pl->scale);
    ++g_launches;
  }
  CUtensorMap mq, mdo, mk0, mv0, mk1, mv1;
  int r;
  if ((r = make_map(&mq, a.q, a.q_tok, pl->h_q, pl->head_dim))) return r;
  if ((r = make_map(&mdo, a.d_o, a.q_tok, pl->h_q, pl->head_dim))) return r;
  if ((r = make_map(&mk0, a.k0, a.kv0_tok, pl->h_kv, pl->head_dim))) return r;
  if ((r = make_map(&mv0, a.v0, a.kv0_tok, pl->h_kv, pl->head_dim))) return r;
  if ((r = make_map(&mk1, a.k1, a.kv1_tok, pl->h_kv, pl->head_dim))) return r;
  if ((r = make_map(&mv1, a.v1, a.kv1_tok, pl->h_kv, pl->head_dim))) return r;
  if (s.n_items() > 0) {
    BwdParams p;
    p.items = s.d_items; p.lane_ptr = s.d_lane_ptr; p.segs = a.d_segs; p.stats = stats;
    p.dk_out = static_cast<__nv_bfloat16 *>(a.dk_out); p.dv_out = static_cast<__nv_bfloat16 *>(a.dv_out);
    p.dk_acc = a.dk_acc; p.dv_acc = a.dv_acc; p.n_tiles = a.n_tiles; p.h_q = pl->h_q; p.h_kv = pl->h_kv; p.d = pl->head_dim;
    p.causal_fp32 = a.causal_fp32; p.scale = pl->scale; p.scale_log2 = pl->scale * 1.4426950408889634f;
    p.status = pl->d_status;
    const int kind = (int)(&s - pl->sched);
    p.wait_budget = wait_budget(pl); p.kind = kind;
    p.test_flags = (pl->flags & AUGTREE_FLAG_TEST_SKIP_BWD_LOAD) ? TEST_SKIP_BWD_LOAD : 0;
    p.no_own = a.no_own;
    p.ds_out = ds; p.pair_tab = reinterpret_cast<const int4 *>(a.d_pairs);
    long long n_run = s.n_items();
    if (a.no_own) {
      n_run = 0;
      for (int i = 0; i < s.n_items(); ++i) n_run += s.items[(size_t)i * s.item_ints + 4] != 0;
    }
    pl->launched_items[kind] += n_run;
    timing_mark(pl, kind, false, st);
    bwd_kernel<D><<<pl->n_lanes, kBwdThreads, BwdSmem<D>::kBytes, st>>>(mq, mdo, mk0, mv0, mk1, mv1, p);
    timing_mark(pl, kind, true, st);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return AUGTREE_ERR_CUDA;
  }
  if (handoff) {
    CUtensorMap mds, mka;
    if ((r = make_ds_map(&mds, ds, a.ds_slots * pl->h_q))) return r;
    if ((r = make_map(&mka, a.ka, a.a_tok, pl->h_kv, pl->head_dim))) return r;
    DqlParams p;
    p.items = a.dq_sched->d_items; p.lane_ptr = a.dq_sched->d_lane_ptr; p.pair_tab = reinterpret_cast<const int4 *>(a.d_pairs);
    p.dq = static_cast<__nv_bfloat16 *>(a.dq); p.dq_f32 = a.dq_f32; p.h_q = pl->h_q; p.d = pl->head_dim; p.no_own = a.no_own;
    p.status = pl->d_status;
    const int kind = (int)(a.dq_sched - pl->sched);
    p.wait_budget = wait_budget(pl); p.kind = kind;
    pl->launched_items[kind] += a.dq_sched->n_items();
    timing_mark(pl, kind, false, st);
    dql_kernel<D><<<pl->n_lanes, kDqlThreads, DqlSmem<D>::kBytes, st>>>(mds, mka, mk0, p);
    timing_mark(pl, kind, true, st);
    ++g_launches;
  } else if (a.dq_sched->n_items() > 0) {
    CUtensorMap mka, mva;
    if ((r = make_map(&mka, a.ka, a.a_tok, pl->h_kv, pl->head_dim))) return r;
    if ((r = make_map(&mva, a.va, a.a_tok, pl->h_kv, pl->head_dim))) return r;
    DqParams p;
    p.items = a.dq_sched->d_items; p.lane_ptr = a.dq_sched->d_lane_ptr; p.stats = stats;
    p.dq = static_cast<__nv_bfloat16 *>(a.dq); p.n_tiles = a.n_tiles; p.h_q = pl->h_q; p.d = pl->head_dim;
    p.scale = pl->scale; p.scale_log2 = pl->scale * 1.4426950408889634f; p.status = pl->d_status;
    const int kind = (int)(a.dq_sched - pl->sched);
    p.wait_budget = wait_budget(pl); p.kind = kind;
    p.no_own = a.no_own; p.dq_f32 = a.dq_f32;
    pl->launched_items[kind] += a.dq_sched->n_items();
    timing_mark(pl, kind, false, st);
    // causal keys come from the queries' own sequence tensor (k0/v0)
    dq_kernel<D><<<pl->n_lanes, kDqThreads, DqSmem<D>::kBytes, st>>>(mq, mdo, mka, mva, mk0, mv0, p);
    timing_mark(pl, kind, true, st);
    ++g_launches;
  }
  return cudaGetLastError() == cudaSuccess ? AUGTREE_OK : AUGTREE_ERR_CUDA;
}

constexpr size_t kTimingPairs = 512;

void timing_mark(const augtree_plan *pl, int kind, bool stop, cudaStream_t st) {
  Timing *t = pl->timing;
  if (!t || !t->on) return;
  size_t &u = t->used[kind];
  if (!stop && u + 2 > t->ev[kind].size()) return;  // pool exhausted: stop recording
  if (stop && (u & 1) == 0) return;
  cudaEventRecord(static_cast<cudaEvent_t>(t->ev[kind][u]), st);
  ++u;
}

// Launch entry points: the plan must live on a device, and that device must be the calling thread's current
// one (tensor maps are encoded and kernels launched in the current context).
int check_plan(const augtree_plan *pl) {
  if (!pl || pl->device < 0 || pl->n_lanes < 1) return AUGTREE_ERR_INVALID_ARG;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) return AUGTREE_ERR_CUDA;
  if (cur != pl->device) return AUGTREE_ERR_INVALID_ARG;
  return AUGTREE_OK;
}

// Queries that only read plan state: any current device will do.
int check_plan_any_device(const augtree_plan *pl) {
  if (!pl || pl->device < 0 || pl->n_lanes < 1) return AUGTREE_ERR_INVALID_ARG;
  return AUGTREE_OK;
}

// The tile kernels use more than the default 48 KB of dynamic shared memory.  The attribute belongs to
// the (function, device) pair, so it is set for the plan's device at plan creation, with that device current.
template <int D>
int set_kernel_attributes() {
  if (cudaFuncSetAttribute(fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<D>::kBytes) != cudaSuccess ||
      cudaFuncSetAttribute(bwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<D>::kBytes) != cudaSuccess ||
      cudaFuncSetAttribute(dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<D>::kBytes) != cudaSuccess ||
      cudaFuncSetAttribute(dql_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqlSmem<D>::kBytes) != cudaSuccess)
    return AUGTREE_ERR_CUDA;
  return AUGTREE_OK;
}

}  // namespace

extern "C" {

int augtree_plan_create(const augtree_desc_t *desc, int device, augtree_plan_t **out) {
  if (!out) return AUGTREE_ERR_INVALID_ARG;
  *out = nullptr;
  if (!desc) return AUGTREE_ERR_INVALID_ARG;
  augtree_plan *pl = new (std::nothrow) augtree_plan();
  if (!pl) return AUGTREE_ERR_INTERNAL;
  augtree_desc_t d = *desc;
  if (device >= 0 && d.struct_size == sizeof(augtree_desc_t) && d.n_lanes == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) {
      delete pl;
      return AUGTREE_ERR_CUDA;
    }
    d.n_lanes = sms;
  }
  if (device < 0 && d.struct_size == sizeof(augtree_desc_t) && d.n_lanes < 1) { delete pl; return AUGTREE_ERR_INVALID_ARG; }
  int r = AUGTREE_ERR_INTERNAL;
  try {
    r = build_plan_host(&d, pl);
  } catch (...) {
    r = AUGTREE_ERR_INTERNAL;
  }
  if (r) { delete pl; return r; }
  pl->device = device;
  if (device >= 0) {
    int prev = 0;
    cudaGetDevice(&prev);
    r = cudaSetDevice(device) == cudaSuccess ? AUGTREE_OK : AUGTREE_ERR_CUDA;
    if (!r) r = pl->head_dim > 64 ? set_kernel_attributes<128>() : set_kernel_attributes<64>();
    try {
      for (int k = 0; k < SCHED_COUNT && !r; ++k)
        r = upload_sched(pl->sched[k], pl->n_lanes, k == SCHED_REPLAY_FWD && (pl->flags & AUGTREE_FLAG_TEST_DROP_ITEM));
    } catch (...) {
      r = AUGTREE_ERR_INTERNAL;
    }
    if (!r) r = upload(pl->seg_replay, &pl->d_seg_replay);
    if (!r) r = upload(pl->seg_prefill, &pl->d_seg_prefill);
    if (!r) r = upload(pl->branch_group, &pl->d_branch_group);
    if (!r) r = upload(pl->group_splits, &pl->d_group_splits);
    if (!r) r = upload(pl->cu_r, &pl->d_cu_r);
    if (!r) r = upload(pl->tiles_replay, &pl->d_tiles_replay);
    if (!r) r = upload(pl->tiles_prefill, &pl->d_tiles_prefill);
    if (!r) r = upload(pl->pairs_replay, &pl->d_pairs_replay);
    if (!r) r = upload(pl->pairs_prefill, &pl->d_pairs_prefill);
    if (!r) {
      if (cudaMalloc(&pl->d_status, kStatusInts * sizeof(int)) != cudaSuccess ||
          cudaMemset(pl->d_status, 0, kStatusInts * sizeof(int)) != cudaSuccess)
        r = AUGTREE_ERR_CUDA;
    }
    cudaSetDevice(prev);
    if (r) { augtree_plan_destroy(pl); return r; }
  }
  *out = pl;
  return AUGTREE_OK;
}

int augtree_plan_destroy(augtree_plan_t *pl) {
  if (!pl) return AUGTREE_ERR_INVALID_ARG;
  if (pl->device >= 0) {
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(pl->device);
    for (int k = 0; k < SCHED_COUNT; ++k) { cudaFree(pl->sched[k].d_items); cudaFree(pl->sched[k].d_lane_ptr); }
    cudaFree(pl->d_seg_replay); cudaFree(pl->d_seg_prefill); cudaFree(pl->d_branch_group); cudaFree(pl->d_group_splits);
    cudaFree(pl->d_cu_r); cudaFree(pl->d_status); cudaFree(pl->d_tiles_replay); cudaFree(pl->d_tiles_prefill);
    cudaFree(pl->d_pairs_replay); cudaFree(pl->d_pairs_prefill);
    if (pl->timing) {
      for (int k = 0; k < SCHED_COUNT; ++k)
        for (void *e : pl->timing->ev[k]) cudaEventDestroy(static_cast<cudaEvent_t>(e));
      delete pl->timing;
    }
    cudaSetDevice(prev);
  }
  delete pl;
  return AUGTREE_OK;
}

int augtree_plan_workspace_bytes(const augtree_plan_t *pl, size_t *fwd, size_t *bwd) {
  if (!pl) return AUGTREE_ERR_INVALID_ARG;
  if (fwd) *fwd = pl->ws_fwd;
  if (bwd) *bwd = pl->ws_bwd;
  return AUGTREE_OK;
}

int augtree_plan_bwd_handoff_bytes(const augtree_plan_t *pl, size_t *bytes) {
  if (!pl || !bytes) return AUGTREE_ERR_INVALID_ARG;
  *bytes = pl->ws_bwd_handoff;
  return AUGTREE_OK;
}

int augtree_plan_metadata(const augtree_plan_t *pl, int table_id, void *host_dst, size_t *bytes) {
  if (!pl || !bytes) return AUGTREE_ERR_INVALID_ARG;
  const std::vector<int32_t> *v = nullptr;
  switch (table_id) {
    case AUGTREE_TBL_CU_PROMPT: v = &pl->cu_p; break;
    case AUGTREE_TBL_CU_BRANCH: v = &pl->cu_b; break;
    case AUGTREE_TBL_CU_RESPONSE: v = &pl->cu_r; break;
    case AUGTREE_TBL_REPLAY_SEGMENTS: v = &pl->seg_replay; break;
    case AUGTREE_TBL_PREFILL_SEGMENTS: v = &pl->seg_prefill; break;
    case AUGTREE_TBL_GROUP_SPLITS: v = &pl->group_splits; break;
    default:
      if (table_id >= AUGTREE_TBL_PREFILL_FWD_ITEMS && table_id <= AUGTREE_TBL_PREFILL_BWD_ORDER) {
        const Sched &s = pl->sched[(table_id - 3) / 3];
        const int which = (table_id - 3) % 3;
        v = which == 0 ? &s.items : which == 1 ? &s.lane_ptr : &s.order;
      } else if (table_id >= AUGTREE_TBL_REPLAY_DQ_ITEMS && table_id <= AUGTREE_TBL_PREFILL_DQ_ORDER) {
        const Sched &s = pl->sched[SCHED_REPLAY_DQ + (table_id - AUGTREE_TBL_REPLAY_DQ_ITEMS) / 3];
        const int which = (table_id - AUGTREE_TBL_REPLAY_DQ_ITEMS) % 3;
        v = which == 0 ? &s.items : which == 1 ? &s.lane_ptr : &s.order;
      }
  }
  if (!v) return AUGTREE_ERR_INVALID_ARG;
  const size_t need = v->size() * sizeof(int32_t);
  if (!host_dst) { *bytes = need; return AUGTREE_OK; }
  if (*bytes < need) { *bytes = need; return AUGTREE_ERR_INVALID_ARG; }
  if (need) std::memcpy(host_dst, v->data(), need);
  *bytes = need;
  return AUGTREE_OK;
}

int augtree_prefill_fwd(const augtree_plan_t *pl, const void *q_p, const void *k_p, const void *v_p, void *o_p,
                        float *lse_p, void *ws, size_t ws_bytes, void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (!q_p || !k_p || !v_p || !o_p || !lse_p) return AUGTREE_ERR_INVALID_ARG;
  if (!aligned16(q_p) || !aligned16(k_p) || !aligned16(v_p) || !aligned16(o_p)) return AUGTREE_ERR_INVALID_ARG;
  if (!ws || ws_bytes < kFwdHeaderBytes || !aligned16(ws)) return AUGTREE_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Sched &s = pl->sched[SCHED_PREFILL_FWD];
  if (pl->head_dim > 64)
    return launch_fwd<128>(pl, s, q_p, pl->total_p, k_p, v_p, pl->total_p, k_p, v_p, pl->total_p, o_p, lse_p, nullptr, nullptr, ws, st);
  return launch_fwd<64>(pl, s, q_p, pl->total_p, k_p, v_p, pl->total_p, k_p, v_p, pl->total_p, o_p, lse_p, nullptr, nullptr, ws, st);
}

int augtree_replay_fwd(const augtree_plan_t *pl, const void *q_r, const void *k_r, const void *v_r, const void *k_p,
                       const void *v_p, void *o_r, float *lse_r, void *ws, size_t ws_bytes, void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (pl->total_r == 0) return AUGTREE_OK;
  if (!q_r || !k_r || !v_r || !k_p || !v_p || !o_r || !lse_r) return AUGTREE_ERR_INVALID_ARG;
  if (!aligned16(q_r) || !aligned16(k_r) || !aligned16(v_r) || !aligned16(k_p) || !aligned16(v_p) || !aligned16(o_r))
    return AUGTREE_ERR_INVALID_ARG;
  float *part_o = nullptr, *part_lse = nullptr;
  if (!ws || ws_bytes < pl->ws_fwd || !aligned16(ws)) return AUGTREE_ERR_WORKSPACE;
  if (pl->max_splits > 1) {
    part_o = reinterpret_cast<float *>(static_cast<uint8_t *>(ws) + kFwdHeaderBytes);
    part_lse = reinterpret_cast<float *>(static_cast<uint8_t *>(ws) + kFwdHeaderBytes +
                                         al256((size_t)pl->max_splits * (size_t)pl->total_r * pl->h_q * pl->head_dim * 4));
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Sched &s = pl->sched[SCHED_REPLAY_FWD];
  if (pl->head_dim > 64)
    r = launch_fwd<128>(pl, s, q_r, pl->total_r, k_p, v_p, pl->total_p, k_r, v_r, pl->total_r, o_r, lse_r, part_o, part_lse, ws, st);
  else
    r = launch_fwd<64>(pl, s, q_r, pl->total_r, k_p, v_p, pl->total_p, k_r, v_r, pl->total_r, o_r, lse_r, part_o, part_lse, ws, st);
  if (r || pl->max_splits == 1) return r;
  // groups that ended up with one shard wrote their final output directly; the
  // merge kernel only touches tokens whose group has more than one shard
  const long long warps = pl->total_r * (long long)pl->h_q;
  const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
  if (pl->head_dim > 64)
    combine_kernel<128><<<blocks, 256, 0, st>>>(part_o, part_lse, pl->d_cu_r, pl->d_branch_group, pl->d_group_splits,
                                                pl->n_branches, static_cast<__nv_bfloat16 *>(o_r), lse_r, pl->total_r, pl->h_q, pl->head_dim);
  else
    combine_kernel<64><<<blocks, 256, 0, st>>>(part_o, part_lse, pl->d_cu_r, pl->d_branch_group, pl->d_group_splits,
                                               pl->n_branches, static_cast<__nv_bfloat16 *>(o_r), lse_r, pl->total_r, pl->h_q, pl->head_dim);
  ++g_launches;
  return cudaGetLastError() == cudaSuccess ? AUGTREE_OK : AUGTREE_ERR_CUDA;
}

// Replay forward without caller scratch: the shard partials live in
// g_static_scratch (file scope, above).  In host code the array's name is only a
// host-side handle, so its device address is looked up once per device, with
// that device current, and handed to the ordinary entry point as its workspace.
int augtree_replay_fwd_static(const augtree_plan_t *pl, const void *q_r, const void *k_r, const void *v_r,
                              const void *k_p, const void *v_p, void *o_r, float *lse_r, void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (pl->ws_fwd > (size_t)AUGTREE_STATIC_SCRATCH_BYTES) return AUGTREE_ERR_WORKSPACE;  // need exceeds the built-in array
  if (pl->device >= kMaxStaticDevices) return AUGTREE_ERR_UNSUPPORTED;
  void *scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[pl->device]) {
      int cur = -1;
      if (cudaGetDevice(&cur) != cudaSuccess) return AUGTREE_ERR_CUDA;
      if (cur != pl->device && cudaSetDevice(pl->device) != cudaSuccess) return AUGTREE_ERR_CUDA;
      void *ptr = nullptr;
      const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
      if (cur != pl->device) cudaSetDevice(cur);
      if (e != cudaSuccess || !ptr) return AUGTREE_ERR_CUDA;
      g_static_ptr[pl->device] = ptr;
    }
    scratch = g_static_ptr[pl->device];
  }
  return augtree_replay_fwd(pl, q_r, k_r, v_r, k_p, v_p, o_r, lse_r, scratch, AUGTREE_STATIC_SCRATCH_BYTES, stream);
}

int augtree_replay_fwd_state(const augtree_plan_t *pl, const void *q_r, const void *k_r, const void *v_r, const void *k_p,
                             const void *v_p, float *state_o, float *state_lse, int include_own, void *ws, size_t ws_bytes,
                             void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (pl->max_splits != 1) return AUGTREE_ERR_UNSUPPORTED;   // a state is one shard's: the plan itself must not shard again
  if (pl->total_r == 0) return AUGTREE_OK;
  if (!q_r || !k_r || !v_r || !k_p || !v_p || !state_o || !state_lse) return AUGTREE_ERR_INVALID_ARG;
  if (!aligned16(q_r) || !aligned16(k_r) || !aligned16(v_r) || !aligned16(k_p) || !aligned16(v_p) || !aligned16(state_o))
    return AUGTREE_ERR_INVALID_ARG;
  if (!ws || ws_bytes < pl->ws_fwd || !aligned16(ws)) return AUGTREE_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Sched &s = pl->sched[SCHED_REPLAY_FWD];
  const int mode = STATE_OUT | (include_own ? 0 : STATE_NO_OWN);
  if (pl->head_dim > 64)
    return launch_fwd<128>(pl, s, q_r, pl->total_r, k_p, v_p, pl->total_p, k_r, v_r, pl->total_r, nullptr, nullptr, state_o, state_lse, ws, st, mode);
  return launch_fwd<64>(pl, s, q_r, pl->total_r, k_p, v_p, pl->total_p, k_r, v_r, pl->total_r, nullptr, nullptr, state_o, state_lse, ws, st, mode);
}

int augtree_merge_states(const augtree_plan_t *pl, int n_states, const float *const *state_o, const float *const *state_lse,
                         void *o_r, float *lse_r, void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (n_states < 1 || n_states > kMaxStates || !state_o || !state_lse || !o_r || !lse_r) return AUGTREE_ERR_INVALID_ARG;
  if (pl->total_r == 0) return AUGTREE_OK;
  StatePtrs sp;
  sp.n = n_states;
  for (int i = 0; i < n_states; ++i) {
    if (!state_o[i] || !state_lse[i]) return AUGTREE_ERR_INVALID_ARG;
    sp.o[i] = state_o[i]; sp.lse[i] = state_lse[i];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const long long warps = pl->total_r * (long long)pl->h_q;
  const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
  if (pl->head_dim > 64)
    merge_states_kernel<128><<<blocks, 256, 0, st>>>(sp, static_cast<__nv_bfloat16 *>(o_r), lse_r, pl->total_r, pl->h_q, pl->head_dim);
  else
    merge_states_kernel<64><<<blocks, 256, 0, st>>>(sp, static_cast<__nv_bfloat16 *>(o_r), lse_r, pl->total_r, pl->h_q, pl->head_dim);
  ++g_launches;
  return cudaGetLastError() == cudaSuccess ? AUGTREE_OK : AUGTREE_ERR_CUDA;
}

int augtree_replay_bwd_state(const augtree_plan_t *pl, const void *q_r, const void *k_r, const void *v_r, const void *k_p,
                             const void *v_p, const void *o_r, const float *lse_r, const void *do_r, float *dq_part, void *dk_r,
                             void *dv_r, float *dkp_acc, float *dvp_acc, int include_own, void *ws, size_t ws_bytes, void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (!dkp_acc || !dvp_acc) return AUGTREE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (pl->flags & AUGTREE_FLAG_ZERO_PROMPT_GRAD) {
    const size_t bytes = (size_t)pl->total_p * pl->h_kv * pl->head_dim * 4;
    if (cudaMemsetAsync(dkp_acc, 0, bytes, st) != cudaSuccess || cudaMemsetAsync(dvp_acc, 0, bytes, st) != cudaSuccess)
      return AUGTREE_ERR_CUDA;
  }
  if (pl->total_r == 0) return AUGTREE_OK;
  if (!q_r || !k_r || !v_r || !k_p || !v_p || !o_r || !lse_r || !do_r || !dq_part) return AUGTREE_ERR_INVALID_ARG;
  if (include_own && (!dk_r || !dv_r)) return AUGTREE_ERR_INVALID_ARG;
  if (!aligned16(q_r) || !aligned16(k_r) || !aligned16(v_r) || !aligned16(k_p) || !aligned16(v_p) || !aligned16(o_r) ||
      !aligned16(do_r) || !aligned16(dq_part) || !aligned16(dk_r) || !aligned16(dv_r) || !aligned16(dkp_acc) || !aligned16(dvp_acc))
    return AUGTREE_ERR_INVALID_ARG;
  if (!ws || ws_bytes < pl->ws_bwd || !aligned16(ws)) return AUGTREE_ERR_WORKSPACE;
  BwdArgs a;
  a.q = q_r; a.d_o = do_r; a.o = o_r; a.lse = lse_r; a.q_tok = pl->total_r;
  a.k0 = k_r; a.v0 = v_r; a.kv0_tok = pl->total_r; a.k1 = k_p; a.v1 = v_p; a.kv1_tok = pl->total_p;
  a.dq = nullptr; a.dk_out = dk_r; a.dv_out = dv_r; a.dk_acc = dkp_acc; a.dv_acc = dvp_acc; a.causal_fp32 = 0;
  a.d_segs = pl->d_seg_replay; a.d_tiles = pl->d_tiles_replay; a.n_tiles = (long long)pl->tiles_replay.size() / 2;
  a.dq_sched = &pl->sched[SCHED_REPLAY_DQ]; a.ka = k_p; a.va = v_p; a.a_tok = pl->total_p;
  a.d_pairs = pl->d_pairs_replay; a.ds_slots = pl->ds_slots_replay;
  a.no_own = include_own ? 0 : 1; a.dq_f32 = dq_part;
  const Sched &s = pl->sched[SCHED_REPLAY_BWD];
  return pl->head_dim > 64 ? launch_bwd<128>(pl, s, a, ws, ws_bytes, st) : launch_bwd<64>(pl, s, a, ws, ws_bytes, st);
}

int augtree_replay_bwd(const augtree_plan_t *pl, const void *q_r, const void *k_r, const void *v_r, const void *k_p,
                       const void *v_p, const void *o_r, const float *lse_r, const void *do_r, void *dq_r, void *dk_r,
                       void *dv_r, float *dkp_acc, float *dvp_acc, void *ws, size_t ws_bytes, void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (!dkp_acc || !dvp_acc) return AUGTREE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (pl->flags & AUGTREE_FLAG_ZERO_PROMPT_GRAD) {
    const size_t bytes = (size_t)pl->total_p * pl->h_kv * pl->head_dim * 4;
    if (cudaMemsetAsync(dkp_acc, 0, bytes, st) != cudaSuccess || cudaMemsetAsync(dvp_acc, 0, bytes, st) != cudaSuccess)
      return AUGTREE_ERR_CUDA;
  }
  if (pl->total_r == 0) return AUGTREE_OK;
  if (!q_r || !k_r || !v_r || !k_p || !v_p || !o_r || !lse_r || !do_r || !dq_r || !dk_r || !dv_r) return AUGTREE_ERR_INVALID_ARG;
  if (!aligned16(q_r) || !aligned16(k_r) || !aligned16(v_r) || !aligned16(k_p) || !aligned16(v_p) || !aligned16(o_r) ||
      !aligned16(do_r) || !aligned16(dq_r) || !aligned16(dk_r) || !aligned16(dv_r) || !aligned16(dkp_acc) || !aligned16(dvp_acc))
    return AUGTREE_ERR_INVALID_ARG;
  if (!ws || ws_bytes < pl->ws_bwd || !aligned16(ws)) return AUGTREE_ERR_WORKSPACE;
  BwdArgs a;
  a.q = q_r; a.d_o = do_r; a.o = o_r; a.lse = lse_r; a.q_tok = pl->total_r;
  a.k0 = k_r; a.v0 = v_r; a.kv0_tok = pl->total_r; a.k1 = k_p; a.v1 = v_p; a.kv1_tok = pl->total_p;
  a.dq = dq_r; a.dk_out = dk_r; a.dv_out = dv_r; a.dk_acc = dkp_acc; a.dv_acc = dvp_acc; a.causal_fp32 = 0;
  a.d_segs = pl->d_seg_replay; a.d_tiles = pl->d_tiles_replay; a.n_tiles = (long long)pl->tiles_replay.size() / 2;
  a.dq_sched = &pl->sched[SCHED_REPLAY_DQ]; a.ka = k_p; a.va = v_p; a.a_tok = pl->total_p;
  a.d_pairs = pl->d_pairs_replay; a.ds_slots = pl->ds_slots_replay;
  const Sched &s = pl->sched[SCHED_REPLAY_BWD];
  return pl->head_dim > 64 ? launch_bwd<128>(pl, s, a, ws, ws_bytes, st) : launch_bwd<64>(pl, s, a, ws, ws_bytes, st);
}

int augtree_prefill_bwd(const augtree_plan_t *pl, const void *q_p, const void *k_p, const void *v_p, const void *o_p,
                        const float *lse_p, const void *do_p, float *dkp_acc, float *dvp_acc, void *dq_p, void *dk_p,
                        void *dv_p, void *ws, size_t ws_bytes, void *stream) {
  int r = check_plan(pl);
  if (r) return r;
  if (!q_p || !k_p || !v_p || !o_p || !lse_p || !do_p || !dkp_acc || !dvp_acc || !dq_p) return AUGTREE_ERR_INVALID_ARG;
  if (!aligned16(q_p) || !aligned16(k_p) || !aligned16(v_p) || !aligned16(o_p) || !aligned16(do_p) || !aligned16(dq_p) ||
      !aligned16(dkp_acc) || !aligned16(dvp_acc) || !aligned16(dk_p) || !aligned16(dv_p))
    return AUGTREE_ERR_INVALID_ARG;
  if (!ws || ws_bytes < pl->ws_bwd || !aligned16(ws)) return AUGTREE_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  BwdArgs a;
  a.q = q_p; a.d_o = do_p; a.o = o_p; a.lse = lse_p; a.q_tok = pl->total_p;
  a.k0 = k_p; a.v0 = v_p; a.kv0_tok = pl->total_p; a.k1 = k_p; a.v1 = v_p; a.kv1_tok = pl->total_p;
  a.dq = dq_p; a.dk_out = nullptr; a.dv_out = nullptr; a.dk_acc = dkp_acc; a.dv_acc = dvp_acc; a.causal_fp32 = 1;
  a.d_segs = pl->d_seg_prefill; a.d_tiles = pl->d_tiles_prefill; a.n_tiles = (long long)pl->tiles_prefill.size() / 2;
  a.dq_sched = &pl->sched[SCHED_PREFILL_DQ]; a.ka = k_p; a.va = v_p; a.a_tok = pl->total_p;
  a.d_pairs = pl->d_pairs_prefill; a.ds_slots = pl->ds_slots_prefill;
  const Sched &s = pl->sched[SCHED_PREFILL_BWD];
  r = pl->head_dim > 64 ? launch_bwd<128>(pl, s, a, ws, ws_bytes, st) : launch_bwd<64>(pl, s, a, ws, ws_bytes, st);
  if (r) return r;
  const long long n4 = pl->total_p * (long long)pl->h_kv * pl->head_dim / 4;
  if (dk_p) { cast_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(dkp_acc, static_cast<__nv_bfloat16 *>(dk_p), n4); ++g_launches; }
  if (dv_p) { cast_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(dvp_acc, static_cast<__nv_bfloat16 *>(dv_p), n4); ++g_launches; }
  return cudaGetLastError() == cudaSuccess ? AUGTREE_OK : AUGTREE_ERR_CUDA;
}

int augtree_last_device_status(const augtree_plan_t *pl, int *status, int *detail) {
  int r = check_plan_any_device(pl);
  if (r || !status) return AUGTREE_ERR_INVALID_ARG;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(pl->device);
  int h[2] = {0, 0};
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(h, pl->d_status, sizeof(h), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && (h[0] || h[1])) e = cudaMemset(pl->d_status, 0, sizeof(h));
  cudaSetDevice(prev);
  if (e != cudaSuccess) return AUGTREE_ERR_CUDA;
  *status = h[0];
  if (detail) *detail = h[1];
  return AUGTREE_OK;
}

int augtree_items_completed(const augtree_plan_t *pl, int kernel, long long *completed, long long *expected) {
  int r = check_plan_any_device(pl);
  if (r || kernel < 0 || kernel >= SCHED_COUNT || !completed || !expected) return AUGTREE_ERR_INVALID_ARG;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(pl->device);
  int n = 0;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(&n, pl->d_status + 2 + kernel, sizeof(int), cudaMemcpyDeviceToHost);
  cudaSetDevice(prev);
  if (e != cudaSuccess) return AUGTREE_ERR_CUDA;
  *completed = n;
  *expected = pl->launched_items[kernel].load();
  return AUGTREE_OK;
}

int augtree_set_timing(augtree_plan_t *pl, int enable) {
  int r = check_plan_any_device(pl);
  if (r) return r;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(pl->device);
  if (!pl->timing) {
    pl->timing = new (std::nothrow) Timing();
    if (!pl->timing) { cudaSetDevice(prev); return AUGTREE_ERR_INTERNAL; }
    for (int k = 0; k < SCHED_COUNT && !r; ++k)
      for (size_t i = 0; i < 2 * kTimingPairs; ++i) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) { r = AUGTREE_ERR_CUDA; break; }
        pl->timing->ev[k].push_back(e);
      }
  }
  pl->timing->on = enable != 0 && !r;
  for (int k = 0; k < SCHED_COUNT; ++k) pl->timing->used[k] = 0;
  cudaSetDevice(prev);
  return r;
}

int augtree_get_kernel_time(const augtree_plan_t *pl, int kernel, float *total_ms, int *launches) {
  int r = check_plan_any_device(pl);
  if (r || kernel < 0 || kernel >= SCHED_COUNT || !total_ms || !launches) return AUGTREE_ERR_INVALID_ARG;
  *total_ms = 0.f; *launches = 0;
  const Timing *t = pl->timing;
  if (!t) return AUGTREE_OK;
  for (size_t i = 0; i + 1 < t->used[kernel]; i += 2) {
    cudaEvent_t a = static_cast<cudaEvent_t>(t->ev[kernel][i]), b = static_cast<cudaEvent_t>(t->ev[kernel][i + 1]);
    if (cudaEventSynchronize(b) != cudaSuccess) return AUGTREE_ERR_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, a, b) != cudaSuccess) return AUGTREE_ERR_CUDA;
    *total_ms += ms;
    ++*launches;
  }
  return AUGTREE_OK;
}

long long augtree_launch_count(void) { return g_launches.load(); }


const char *augtree_status_string(int s) {
  switch (s) {
    case AUGTREE_OK: return "ok";
    case AUGTREE_ERR_INVALID_ARG: return "invalid argument";
    case AUGTREE_ERR_UNSUPPORTED: return "unsupported configuration";
    case AUGTREE_ERR_WORKSPACE: return "workspace missing or too small";
    case AUGTREE_ERR_CUDA: return "CUDA call failed";
    case AUGTREE_ERR_TIMEOUT: return "device-side wait timed out";
    case AUGTREE_ERR_INTERNAL: return "internal error";
    default: return "unknown status";
  }
}

}  // extern "C"
