/*
 * augtree.h -- C interface of the prompt-sharing tree-attention library for
 * NVIDIA B200 (sm_100a).
 *
 * The library computes, on one GPU, the attention part of the update-stage
 * replay of a batch of prompt-response trees T = (P, {R_i}, i = 1..G)
 * (Sec. 3.1 of the paper): one causal prefill of every shared prompt, the
 * replay of every response branch against [shared prompt KV | own causal
 * response KV] (Eq. 1), and the exact backward pass in which the prompt KV
 * gradient is the sum over all branches (Eq. 2) and is then carried back
 * through the prefill.
 *
 * Conventions that hold for every entry point
 *  - Tensors are DEVICE pointers owned by the caller, bf16 unless stated,
 *    laid out [tokens, heads, head_dim] with head_dim contiguous.  Prompt
 *    tokens of all groups are packed back to back in group order; response
 *    tokens are packed group-major, then branch order.  No padding, no
 *    alignment requirement on the lengths; base pointers 16-byte aligned.
 *  - LSE tensors are fp32 [H_q, tokens]: natural log of the sum of
 *    exponentials of the scaled scores (m + ln l of the (m, l, O_acc) state of
 *    Sec. 3.3).
 *  - Query head h reads KV head h / (H_q / H_kv).
 *  - Row a of a sequence sees keys b <= a (inclusive diagonal).
 *  - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous; they
 *    return after enqueueing.  Nothing is allocated or freed per call.
 *  - A plan belongs to the device given to augtree_plan_create.  The five
 *    launching entry points (prefill/replay, fwd/bwd, and the static-scratch
 *    forward) must be called with that device current in the calling thread
 *    and with a stream of that device; with another device current they
 *    return AUGTREE_ERR_INVALID_ARG and launch nothing.  One process may hold
 *    plans for several devices and use them from several threads; a plan is
 *    immutable after creation, and concurrent calls on one plan are safe as
 *    long as each has its own workspace.  Plan creation, destruction and the
 *    status and timing queries switch to the plan's device themselves and
 *    restore the caller's.
 *  - Every function returns AUGTREE_OK (0) or a negative augtree_status code;
 *    the library never aborts, traps or throws.  Errors detected on the
 *    device (a bounded wait that ran out) are recorded in a status word that
 *    augtree_last_device_status reads back.
 *  - The descriptor arrays are HOST memory and are only read during
 *    augtree_plan_create.
 */
#ifndef AUGTREE_H_
#define AUGTREE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AUGTREE_VERSION 1u

typedef enum {
  AUGTREE_OK = 0,
  AUGTREE_ERR_INVALID_ARG = -1, /* null pointer, non-positive length, bad struct size   */
  AUGTREE_ERR_UNSUPPORTED = -2, /* head_dim unsupported, h_q % h_kv != 0, sizes too big */
  AUGTREE_ERR_WORKSPACE = -3,   /* workspace pointer null or too small                  */
  AUGTREE_ERR_CUDA = -4,        /* a CUDA runtime or driver call failed                 */
  AUGTREE_ERR_TIMEOUT = -5,     /* a device-side wait gave up (status word)             */
  AUGTREE_ERR_INTERNAL = -6
} augtree_status;

/* flags */
#define AUGTREE_FLAG_ZERO_PROMPT_GRAD 1u /* replay_bwd clears dkp_acc/dvp_acc before accumulating */
/*
 * Fault injection for tests of the failure paths.  The faults are made on the
 * host or by leaving work undone; none of them faults, traps or hangs the
 * device, and a plan without these flags behaves as if they did not exist.
 *  SHORT_WAIT     every device-side wait gives up after about a millisecond
 *                 instead of about a second
 *  SKIP_FWD_LOAD  lane 0 of the forward kernels never loads the first V tile of
 *                 its first item: the wait for it runs out, the lane records
 *                 AUGTREE_ERR_TIMEOUT and returns; the other lanes finish
 *  SKIP_BWD_LOAD  the same for the first dO tile of the key-side backward kernel
 *  DROP_ITEM      the device copy of the replay-forward lane table loses one
 *                 item; augtree_items_completed then reports the shortfall
 */
#define AUGTREE_FLAG_TEST_SHORT_WAIT 0x100u
#define AUGTREE_FLAG_TEST_SKIP_FWD_LOAD 0x200u
#define AUGTREE_FLAG_TEST_SKIP_BWD_LOAD 0x400u
#define AUGTREE_FLAG_TEST_DROP_ITEM 0x800u

/*
 * Packed group descriptor (host, plain data).  One entry per replay tree
 * ("group"): its prompt length P_g >= 1, its branch count G_g >= 0 and, in
 * branch_len, the G_g response lengths R_{g,i} >= 1 of every group one after
 * another (Sec. 3.1: T = (P, {R_i})).  G_g = 0 describes a prompt with no
 * responses; a batch of such groups is the flattened no-reuse baseline when
 * each "prompt" is one linear sequence [P; R_i] (the ordinary causal pass of
 * Sec. 3.4, b = 0).
 */
typedef struct {
  uint32_t struct_size;       /* sizeof(augtree_desc_t)                                  */
  uint32_t version;           /* AUGTREE_VERSION                                         */
  int32_t n_groups;
  const int32_t *prompt_len;  /* [n_groups]                                       (host) */
  const int32_t *n_branches;  /* [n_groups]                                       (host) */
  const int32_t *branch_len;  /* [sum n_branches], group-major                    (host) */
  int32_t h_q, h_kv, head_dim;/* multiple of 8, 8..128; tiles are 64 or 128 wide      */
  float softmax_scale;        /* 0 => 1/sqrt(head_dim)  (Sec. 2.2)                       */
  uint32_t flags;
  int32_t n_lanes;            /* replay lanes = persistent CTAs; 0 => SM count of device */
  int32_t kv_splits;          /* prompt-KV shards per query tile in replay_fwd; 0/1 none */
} augtree_desc_t;

typedef struct augtree_plan augtree_plan_t;

/* Tables returned by augtree_plan_metadata (all int32). */
enum {
  AUGTREE_TBL_CU_PROMPT = 0,      /* [n_groups+1] prefix sums of prompt_len                 */
  AUGTREE_TBL_CU_BRANCH = 1,      /* [n_groups+1] prefix sums of n_branches                 */
  AUGTREE_TBL_CU_RESPONSE = 2,    /* [n_branches+1] prefix sums of branch_len               */
  AUGTREE_TBL_PREFILL_FWD_ITEMS = 3, AUGTREE_TBL_PREFILL_FWD_LANE_PTR = 4, AUGTREE_TBL_PREFILL_FWD_ORDER = 5,
  AUGTREE_TBL_REPLAY_FWD_ITEMS = 6,  AUGTREE_TBL_REPLAY_FWD_LANE_PTR = 7,  AUGTREE_TBL_REPLAY_FWD_ORDER = 8,
  AUGTREE_TBL_REPLAY_BWD_ITEMS = 9,  AUGTREE_TBL_REPLAY_BWD_LANE_PTR = 10, AUGTREE_TBL_REPLAY_BWD_ORDER = 11,
  AUGTREE_TBL_PREFILL_BWD_ITEMS = 12, AUGTREE_TBL_PREFILL_BWD_LANE_PTR = 13, AUGTREE_TBL_PREFILL_BWD_ORDER = 14,
  AUGTREE_TBL_REPLAY_SEGMENTS = 15,  /* [n_branches][3] {first response token, length, first query-tile index} */
  AUGTREE_TBL_PREFILL_SEGMENTS = 16, /* [n_groups][3]   {first prompt token, length, first query-tile index}   */
  AUGTREE_TBL_GROUP_SPLITS = 17,     /* [n_groups] prompt-KV shards actually used           */
  AUGTREE_TBL_REPLAY_DQ_ITEMS = 18,  AUGTREE_TBL_REPLAY_DQ_LANE_PTR = 19,  AUGTREE_TBL_REPLAY_DQ_ORDER = 20,
  AUGTREE_TBL_PREFILL_DQ_ITEMS = 21, AUGTREE_TBL_PREFILL_DQ_LANE_PTR = 22, AUGTREE_TBL_PREFILL_DQ_ORDER = 23,
  AUGTREE_TBL_COUNT = 24
};
#define AUGTREE_FWD_ITEM_INTS 12
#define AUGTREE_BWD_ITEM_INTS 8

/*
 * Pack and schedule (host).  Validates the descriptor, builds the prefix sums
 * and, for each of the six schedules (forward, key-side and query-side
 * backward, each for the prefill and the replay call), the list of work items and their
 * assignment to `n_lanes` replay lanes: items weighted by their valid Q-KV
 * tile count are placed largest first on the least loaded lane (the balanced
 * makespan assignment of Sec. 3.4, Eq. 6, in its greedy form with one round).
 * With device >= 0 the tables are also copied to that device and a status
 * word is allocated there; with device < 0 the plan is host-only (metadata
 * queries work, launches return AUGTREE_ERR_INVALID_ARG) and n_lanes must be
 * given.  This is the only entry point, with augtree_plan_destroy, that
 * allocates or frees device memory.
 */
int augtree_plan_create(const augtree_desc_t *desc, int device, augtree_plan_t **out);
int augtree_plan_destroy(augtree_plan_t *plan);

/*
 * Bytes of caller-provided scratch the forward and backward calls need.  Both
 * forward calls need at least 256 bytes (the largest key norm per KV head,
 * from which the tile kernel bounds the scores of a row), the sharded replay
 * forward also room for the shards' partial states; the backward calls need
 * the per-row statistics.
 */
int augtree_plan_workspace_bytes(const augtree_plan_t *plan, size_t *fwd_bytes, size_t *bwd_bytes);

/*
 * Backward scratch size from which the backward calls take the hand-off path.  The textbook backward of
 * attention is five GEMMs per (query tile, KV tile) pair; with bwd_bytes of scratch the two kernels of a
 * backward call (key side: dK, dV; query side: dQ) each recompute S and dP, seven GEMMs in all.  A call
 * given ws_bytes >= *bytes instead has the key-side kernel store dS (bf16, 32 KB per pair and query head:
 * *bytes = bwd_bytes + that, the larger of the two backward calls) and the query-side kernel compute
 * dQ = sum dS K from it: five GEMMs, at the price of writing and reading the scratch once.  Both paths give
 * dK, dV bit for bit the same.  dQ then comes from the very dS values that went into dK instead of the query-side
 * kernel's own recomputation of them (whose bf16 rounding of dS falls differently on a few per cent of the
 * elements): the two paths' dQ agree to one bf16 step.  *bytes is
 * SIZE_MAX for a plan too large to index; the choice is the caller's, per call, through ws_bytes.  The path also
 * needs ws aligned to 32 bytes (the tiles are written with 32-byte stores); a less aligned ws takes the recomputing
 * path whatever its size.
 */
int augtree_plan_bwd_handoff_bytes(const augtree_plan_t *plan, size_t *bytes);

/*
 * Copy one metadata table to host memory.  With host_dst == NULL only *bytes
 * is set.  Otherwise *bytes is the capacity on entry and the size on return.
 * Item layouts (int32 each):
 *   forward item  [12]: q_tok0, q_pos0, q_rows, q_head, a_tok0, a_len, b_tok0,
 *                       b_len, split, n_splits, weight, kv_head
 *     a_* : unmasked key range (shared prompt KV, Eq. 1's KV_P), b_* : causal
 *     key range of the query's own sequence, length already clipped to what
 *     the tile's last row sees.
 *   backward item [8] : kv_tok0, kv_pos0, kv_rows, kv_head, mode, seg0, nseg,
 *                       weight;  mode 0 = causal inside one sequence, mode 1 =
 *     shared prompt keys against every response query of the group (Eq. 2).
 *     These are the units of the key-side backward kernel (dK, dV).
 *   dQ item [12]: a forward item that is never sharded; field 8 holds the
 *     index of the query tile (segment's first tile index + tile) instead of
 *     the shard number.  Units of the query-side backward kernel.
 *   *_LANE_PTR [n_lanes+1], *_ORDER [n_items]: lane l runs the items
 *     ORDER[LANE_PTR[l] .. LANE_PTR[l+1]) in that order.
 */
int augtree_plan_metadata(const augtree_plan_t *plan, int table_id, void *host_dst, size_t *bytes);

/*
 * Prompt prefill, forward (Sec. 3.2, "Shared prompt prefill pass"): causal
 * attention of every prompt on itself.  k_p/v_p are only read and stay where
 * they are for the replay calls.
 *   q_p [sumP,H_q,d]  k_p,v_p [sumP,H_kv,d]  ->  o_p [sumP,H_q,d] bf16, lse_p [H_q,sumP] fp32
 * ws: fwd_bytes of scratch (augtree_plan_workspace_bytes), else AUGTREE_ERR_WORKSPACE.
 */
int augtree_prefill_fwd(const augtree_plan_t *plan, const void *q_p, const void *k_p, const void *v_p,
                        void *o_p, float *lse_p, void *ws, size_t ws_bytes, void *stream);

/*
 * Response replay, forward (Sec. 3.2 "Response replay", Sec. 3.3): every
 * response query attends to the shared prompt KV (unmasked) and to its own
 * branch (causal); the partial softmax states of the parts are merged
 * (the (+) of Sec. 3.3).  With kv_splits > 1 the prompt KV of a query tile is
 * processed as independent shards whose states are merged by a second kernel.
 *   q_r [sumR,H_q,d] k_r,v_r [sumR,H_kv,d] k_p,v_p -> o_r [sumR,H_q,d] bf16, lse_r [H_q,sumR] fp32
 */
int augtree_replay_fwd(const augtree_plan_t *plan, const void *q_r, const void *k_r, const void *v_r,
                       const void *k_p, const void *v_p, void *o_r, float *lse_r,
                       void *ws, size_t ws_bytes, void *stream);

/*
 * Response replay, backward (Sec. 3.2, "Exact many-to-one backward", Eq. 2).
 * Inputs as the forward plus its outputs o_r, lse_r and the seed do_r.
 * Outputs dq_r [sumR,H_q,d], dk_r, dv_r [sumR,H_kv,d] bf16.  The prompt-KV
 * gradients of all branches and query heads are ADDED into the fp32
 * accumulators dkp_acc, dvp_acc [sumP,H_kv,d], which the caller zeroes first
 * (or sets AUGTREE_FLAG_ZERO_PROMPT_GRAD in the descriptor).  Each prompt-KV
 * tile is owned by one lane, so this sum has a fixed order; dq_r comes from a
 * second, query-stationary kernel in which each query tile has one owner.
 * No atomics are used: results are bitwise repeatable.
 */
int augtree_replay_bwd(const augtree_plan_t *plan, const void *q_r, const void *k_r, const void *v_r,
                       const void *k_p, const void *v_p, const void *o_r, const float *lse_r,
                       const void *do_r, void *dq_r, void *dk_r, void *dv_r,
                       float *dkp_acc, float *dvp_acc, void *ws, size_t ws_bytes, void *stream);

/*
 * Prompt prefill, backward: the causal backward of augtree_prefill_fwd under
 * the seed do_p.  Its dK/dV are ADDED to dkp_acc/dvp_acc, which after this
 * call hold the final prompt-KV gradients (replay seeds + prefill graph,
 * Sec. 3.2); call it after augtree_replay_bwd on the same stream.  dq_p is
 * written; dk_p/dv_p (bf16 copies of the final accumulators) may be NULL,
 * and then the two backward calls may come in either order: each adds its
 * terms of the same sum to the fp32 accumulators.
 */
int augtree_prefill_bwd(const augtree_plan_t *plan, const void *q_p, const void *k_p, const void *v_p,
                        const void *o_p, const float *lse_p, const void *do_p,
                        float *dkp_acc, float *dvp_acc, void *dq_p, void *dk_p, void *dv_p,
                        void *ws, size_t ws_bytes, void *stream);

/*
 * augtree_replay_fwd for callers that cannot hand the library a scratch
 * buffer.  (The paper has no counterpart: this is a packaging variant of the
 * sharded replay forward, not a step of the method.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a
 * plug-in inside a host runtime that owns the allocator and only passes in
 * pre-existing tensors, a real-time loop that must not take the allocator
 * lock, a process whose memory is fully pre-partitioned.  Such a caller can
 * point at its inputs and outputs but cannot obtain the `ws` block that the
 * sharded forward needs for the per-shard partial softmax states.
 *
 * Here that scratch is a fixed array inside the library's device image,
 * AUGTREE_STATIC_SCRATCH_BYTES (32 MiB) large.  Every GPU on which the
 * library's code is loaded keeps those 32 MiB reserved until the process
 * exits, whether or not this function is ever called.  The call performs no
 * cudaMalloc / cudaFree and uses no allocating library routine; the plan must
 * already exist (augtree_plan_create is the allocating step and belongs to
 * set-up).
 *
 *  - A plan whose forward scratch need (augtree_plan_workspace_bytes, fwd)
 *    exceeds the array is refused with AUGTREE_ERR_WORKSPACE; nothing is
 *    launched.  Plans without prompt-KV shards need 256 bytes and always fit.
 *  - The first call on each device looks up the array's device address (a
 *    one-off set-up step, done with that device current).  Make that first
 *    call outside any stream capture.
 *  - All calls on a device share the one array and it keeps whatever the last
 *    call left there.  The one part that must start at zero (the key-norm
 *    maxima at its head, when several blocks combine them) is cleared by the
 *    call itself on its stream; every other value read is written by the same
 *    call first.  Two
 *    calls that may overlap on the GPU (different streams, no dependency) race
 *    on it; order them.
 * Arguments and results are those of augtree_replay_fwd.
 */
#define AUGTREE_STATIC_SCRATCH_BYTES (32u << 20)
int augtree_replay_fwd_static(const augtree_plan_t *plan, const void *q_r, const void *k_r, const void *v_r,
                              const void *k_p, const void *v_p, void *o_r, float *lse_r, void *stream);

/*
 * Synchronises the plan's device and reads the device status word: *status is
 * AUGTREE_OK or AUGTREE_ERR_TIMEOUT; *detail (may be NULL) gets a code that
 * names the wait that gave up.  The word is cleared by the read.
 */
int augtree_last_device_status(const augtree_plan_t *plan, int *status, int *detail);

/*
 * Building blocks of context-parallel replay (Sec. 3.3 "Common tile semantics", MoveQ and TreeMoveKV).  A rank
 * that holds one shard of the keys computes, for every response query it is given, the PARTIAL online-softmax
 * state over that shard; the states of a query are merged afterwards (the (+) of Sec. 3.3), on whichever rank
 * owns the query; in the backward pass every shard owner computes its shard's dK, dV and its contribution to dQ
 * from the merged LSE, and the dQ contributions are summed on the way back (in the backward pass of MoveQ the
 * exchange of the forward pass runs in reverse, Sec. 3.3).  These three calls are the per-rank compute steps; moving queries,
 * states and gradients between ranks is the caller's (NCCL or peer copies, no multicast loads).  state_o,
 * state_lse and dq_part are written with plain global stores from the tile kernels' epilogues, so they may be
 * peer-mapped memory of the rank that will merge them: the exchange then happens as the tiles finish.  Inputs
 * are read through TMA and must be this device's own memory.
 *
 * The plan describes THIS RANK'S view: its "prompt" is the shard of unmasked keys it holds (k_p, v_p: a prompt-KV
 * shard, or any keys every given query may see in full), its branches are the response queries it is given.
 * The plan must not use kv_splits.
 *
 * augtree_replay_fwd_state: state_o [sumR,H_q,d] fp32 (normalised partial output) and state_lse [H_q,sumR] fp32
 *   over the keys {the plan's prompt} and, if include_own != 0, the query's own causal response prefix (k_r, v_r).
 *   The state is kept as (normalised O, LSE): the same information as (m, l, O_acc).
 * augtree_merge_states: merges n_states <= 16 such states (HOST arrays of DEVICE pointers) into o_r (bf16) and
 *   lse_r; a state whose LSE is -inf (no key seen) has weight zero.  The states are read with plain global loads,
 *   once each, so the pointers may also be peer-mapped memory of the ranks that computed them: the gather of
 *   the states and their merge are then one kernel.
 * augtree_replay_bwd_state: with the MERGED o_r, lse_r and the seed do_r: dkp_acc, dvp_acc += gradients of the
 *   plan's prompt keys over all given queries (complete for this shard: Eq. 2's sum is local to the shard's owner);
 *   dq_part [sumR,H_q,d] fp32 = this shard's contribution to dQ (written, not added); with include_own != 0 also
 *   the own-response part: dk_r, dv_r (bf16) written and the causal range included in dq_part; with
 *   include_own == 0, dk_r and dv_r may be NULL, and k_r, v_r are not read (they must still be valid device
 *   pointers of the plan's response shape: a tensor map is encoded over them).
 */
int augtree_replay_fwd_state(const augtree_plan_t *plan, const void *q_r, const void *k_r, const void *v_r,
                             const void *k_p, const void *v_p, float *state_o, float *state_lse, int include_own,
                             void *ws, size_t ws_bytes, void *stream);
int augtree_merge_states(const augtree_plan_t *plan, int n_states, const float *const *state_o,
                         const float *const *state_lse, void *o_r, float *lse_r, void *stream);
int augtree_replay_bwd_state(const augtree_plan_t *plan, const void *q_r, const void *k_r, const void *v_r,
                             const void *k_p, const void *v_p, const void *o_r, const float *lse_r, const void *do_r,
                             float *dq_part, void *dk_r, void *dv_r, float *dkp_acc, float *dvp_acc, int include_own,
                             void *ws, size_t ws_bytes, void *stream);

/*
 * Work accounting (no counterpart in the paper's method).  Every tile kernel
 * counts the work items it has finished; the host counts the items it has
 * handed to launches.  Synchronises the plan's device and returns both counts
 * for one kernel (numbering as in augtree_get_kernel_time), summed over the
 * plan's lifetime.  completed < expected after a synchronised call means that
 * some lane did not run or did not finish an item (a lane that gave up on a
 * wait, a damaged lane table): its outputs are stale.
 */
int augtree_items_completed(const augtree_plan_t *plan, int kernel, long long *completed, long long *expected);

/*
 * Measurement aid (no counterpart in the paper's method; Sec. 4.1 reports such
 * per-kernel attention times).  With enable != 0 every later launch of the four
 * tile kernels on this plan is bracketed by a pair of CUDA events recorded on
 * the launch's stream (up to 512 launches per kernel, then recording stops);
 * each call resets the record.  The events are created on the first call,
 * which is therefore not free; the launches themselves stay asynchronous.
 * augtree_get_kernel_time waits for the recorded launches of one kernel
 * (0 prefill fwd, 1 replay fwd, 2 replay bwd dK/dV, 3 prefill bwd dK/dV, 4 replay bwd dQ,
 * 5 prefill bwd dQ) and returns their
 * summed device time and count.
 */
int augtree_set_timing(augtree_plan_t *plan, int enable);
int augtree_get_kernel_time(const augtree_plan_t *plan, int kernel, float *total_ms, int *launches);

/* Number of kernel launches the library has enqueued since it was loaded. */
long long augtree_launch_count(void);

/*
 * Replay-grid assignment (Sec. 3.4 "Replay units and grid assignment", Eq. 6; the AssignGrid step of
 * Algorithm 1).  Host only, no device work.  n_units replay units with work weight[k] >= 0 and size
 * size[k] >= 0 are placed on a grid of n_rounds x n_lanes cells, unit k into cell (round_out[k],
 * lane_out[k]).  Lanes of a round run concurrently and rounds run in sequence, so the predicted
 * critical path is  sum over rounds of (max over lanes of (sum of the weights placed there)),  which
 * is what is minimised and returned in *critical_path; a cell holds at most cell_cap of size
 * (cell_cap <= 0: no limit, size may then be NULL).  Up to exact_max_units units (0 selects 12, at
 * most 16) the minimum is exact (dynamic programming over subsets) and *solved_exactly is 1; above
 * it units are placed largest first (ties: lower index), each into the cell that fits and lengthens
 * the path least, then the lightest such cell, then the lowest round, then the lowest lane, and
 * *solved_exactly is 0.  All arrays are host memory owned by the caller; critical_path and
 * solved_exactly may be NULL.  Returns AUGTREE_ERR_INVALID_ARG for bad arguments and
 * AUGTREE_ERR_UNSUPPORTED when the units cannot be packed under cell_cap (exact solver: no packing
 * exists; greedy: none was found) or the grid is larger than 1024 rounds x 65536 lanes.
 */
int augtree_assign_grid(const int64_t *weight, const int64_t *size, int n_units, int n_rounds, int n_lanes,
                        int64_t cell_cap, int exact_max_units, int32_t *round_out, int32_t *lane_out,
                        int64_t *critical_path, int32_t *solved_exactly);

/*
 * Online strategy planner (Sec. 3.4 "Online Strategy Planner", Algorithm 1, Eq. 6-10).  Host only, no device work.
 * For one replay tree T = (P, {R_i}) and a set of candidate CP degrees it enumerates the candidates
 * c = (d, pi, (b, s), X): per degree d the fused candidate (RingCP, b = 0: ordinary ring CP over every (P, R_i) pair,
 * the prompt recomputed per branch) and, for pi in {TreeMoveKV, MoveQ}, every lane count s that divides d (s <= G) and
 * every round count b = 1 .. min(b_max, ceil(G / s)).  The replay units are the G response paths, unit k with weight
 * w_k = its valid Q-KV tile count in replay (128 x 128 tiles: query tiles x prompt tiles + its causal triangle) and size
 * R_k tokens; X comes from the AssignGrid step (augtree_assign_grid: exact up to exact_max_units units, largest-first
 * above) under the cell limit the memory model gives.  Each feasible candidate is scored with Eq. 7,
 *   T(c) = gamma_c (T_prefill + T_replay),
 *   Eq. 8   T_prefill = alpha_p L_P / d_eff + beta_p L_P f_ring(d_eff) + lat_p0 + lat_p1 d_eff
 *           (d_eff = d for MoveQ; d_lane = d / s for TreeMoveKV, where every lane prefills the prompt itself),
 *   Eq. 9   TreeMoveKV: alpha_tmkv W / d_lane + beta_tmkv C_KV + lat_tmkv0 + lat_tmkv1 b d_lane,
 *           C_KV = b 2 (L_P + L_cell) H_kv f_ring(d_lane)                                        (Eq. 3 per round),
 *   Eq. 10  MoveQ: alpha_mq W / d_lane + beta_q C_Q + T_r + lat_mq0 + lat_mq1 b,
 *           C_Q = b L_cell H_q (Eq. 4),  T_r = b (red0 + red1 L_cell H_q) f_ring(d),
 *   b = 0   gamma_ring sum_i [alpha_ring tiles(L_P + R_i) / d + beta_ring 2 (L_P + R_i) H_kv f_ring(d) + lat_ring0 + lat_ring1 d],
 * with W the critical-path work of X (Eq. 6's objective), f_ring(d) = (d - 1) / d, and L_cell = ceil(G / (b s)) max_i R_i,
 * the paper's conservative replay-length proxy applied to a cell.  Per-rank memory (mem_cap <= 0: no limit):
 * TreeMoveKV  mem_prompt L_P / d_lane + mem_resp cell_tokens / d_lane <= mem_cap;  MoveQ  mem_prompt L_P / d +
 * mem_resp cell_tokens / d_lane <= mem_cap;  RingCP  (mem_prompt L_P + mem_resp max_i R_i) / d <= mem_cap.
 * The paper gives the form of these terms and leaves every constant to profiling, so all constants are inputs; the
 * definitions of f_ring, L_cell, T_r and the memory shares are this library's readings of what the paper leaves open.
 * Ties go to the candidate enumerated first (degrees in the given order, RingCP, TreeMoveKV, MoveQ, s ascending, b
 * ascending).  round_out / lane_out [n_branches] receive X of the chosen candidate (zeros for RingCP).  Returns
 * AUGTREE_ERR_UNSUPPORTED when no candidate is feasible.  All pointers are host memory owned by the caller.
 */
enum { AUGTREE_RING_CP = 0, AUGTREE_TREE_MOVE_KV = 1, AUGTREE_MOVE_Q = 2 };
typedef struct {
  double alpha_p, beta_p, lat_p0, lat_p1;
  double alpha_tmkv, beta_tmkv, lat_tmkv0, lat_tmkv1;
  double alpha_mq, beta_q, red0, red1, lat_mq0, lat_mq1;
  double alpha_ring, beta_ring, lat_ring0, lat_ring1;
  double gamma_ring, gamma_tmkv, gamma_mq;
  double mem_cap, mem_prompt, mem_resp;
} augtree_profile_t;
typedef struct {
  uint32_t struct_size;        /* sizeof(augtree_tree_t)                                  */
  int32_t prompt_len;          /* L_P >= 1                                                */
  int32_t n_branches;          /* G >= 0                                                  */
  const int32_t *branch_len;   /* [G] R_i >= 1                                     (host) */
  int32_t h_q, h_kv;
  int32_t n_degrees;
  const int32_t *degrees;      /* [n_degrees] candidate CP degrees d >= 1          (host) */
  int32_t b_max;               /* most rounds tried; 0 selects 4                          */
  int32_t exact_max_units;     /* as in augtree_assign_grid; 0 selects 12                 */
} augtree_tree_t;
typedef struct {
  double cost;                 /* T(c*) by Eq. 7                                          */
  int32_t degree, primitive, rounds, lanes;   /* d, pi, b, s of c*                        */
  int32_t solved_exactly;      /* 1: X of c* is an exact minimum of Eq. 6                 */
  int32_t n_candidates;        /* candidates enumerated                                   */
} augtree_choice_t;
int augtree_plan_tree(const augtree_tree_t *tree, const augtree_profile_t *profile, augtree_choice_t *choice,
                      int32_t *round_out, int32_t *lane_out);

const char *augtree_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* AUGTREE_H_ */
