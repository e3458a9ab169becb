"""ctypes binding of libaugtree.so: argument marshalling only.

Every step of the path runs inside the library's kernels.  PyTorch appears only
as the owner of device memory and of the current stream.  Importing this module
raises if the library has not been built (there is no CPU fallback):
run `python -m paper_2609_33133_b200.build`.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AUGTREE_LIB") or os.path.join(_HERE, "libaugtree.so")   # AUGTREE_LIB: another build of the library
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_33133_b200.build`")
lib = C.CDLL(LIB_PATH)

FLAG_ZERO_PROMPT_GRAD = 1
FLAG_TEST_SHORT_WAIT, FLAG_TEST_SKIP_FWD_LOAD, FLAG_TEST_SKIP_BWD_LOAD, FLAG_TEST_DROP_ITEM = 0x100, 0x200, 0x400, 0x800
STATIC_SCRATCH_BYTES = 32 << 20
FWD_ITEM_INTS, BWD_ITEM_INTS = 12, 8
(TBL_CU_PROMPT, TBL_CU_BRANCH, TBL_CU_RESPONSE, TBL_PREFILL_FWD_ITEMS, TBL_PREFILL_FWD_LANE_PTR, TBL_PREFILL_FWD_ORDER,
 TBL_REPLAY_FWD_ITEMS, TBL_REPLAY_FWD_LANE_PTR, TBL_REPLAY_FWD_ORDER, TBL_REPLAY_BWD_ITEMS, TBL_REPLAY_BWD_LANE_PTR,
 TBL_REPLAY_BWD_ORDER, TBL_PREFILL_BWD_ITEMS, TBL_PREFILL_BWD_LANE_PTR, TBL_PREFILL_BWD_ORDER, TBL_REPLAY_SEGMENTS,
 TBL_PREFILL_SEGMENTS, TBL_GROUP_SPLITS, TBL_REPLAY_DQ_ITEMS, TBL_REPLAY_DQ_LANE_PTR, TBL_REPLAY_DQ_ORDER,
 TBL_PREFILL_DQ_ITEMS, TBL_PREFILL_DQ_LANE_PTR, TBL_PREFILL_DQ_ORDER) = range(24)

EXPORTS = ["augtree_plan_create", "augtree_plan_destroy", "augtree_plan_workspace_bytes", "augtree_plan_metadata",
           "augtree_prefill_fwd", "augtree_replay_fwd", "augtree_replay_bwd", "augtree_prefill_bwd",
           "augtree_last_device_status", "augtree_launch_count", "augtree_status_string",
           "augtree_set_timing", "augtree_get_kernel_time", "augtree_replay_fwd_static", "augtree_assign_grid",
           "augtree_items_completed", "augtree_plan_tree", "augtree_replay_fwd_state", "augtree_merge_states",
           "augtree_replay_bwd_state", "augtree_plan_bwd_handoff_bytes"]


class Desc(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("version", C.c_uint32), ("n_groups", C.c_int32),
                ("prompt_len", C.POINTER(C.c_int32)), ("n_branches", C.POINTER(C.c_int32)),
                ("branch_len", C.POINTER(C.c_int32)), ("h_q", C.c_int32), ("h_kv", C.c_int32),
                ("head_dim", C.c_int32), ("softmax_scale", C.c_float), ("flags", C.c_uint32),
                ("n_lanes", C.c_int32), ("kv_splits", C.c_int32)]


_vp, _sz = C.c_void_p, C.c_size_t
_i64p, _i32p = C.POINTER(C.c_int64), C.POINTER(C.c_int32)
lib.augtree_plan_create.argtypes = [C.POINTER(Desc), C.c_int, C.POINTER(_vp)]
lib.augtree_plan_destroy.argtypes = [_vp]
lib.augtree_plan_workspace_bytes.argtypes = [_vp, C.POINTER(_sz), C.POINTER(_sz)]
lib.augtree_plan_bwd_handoff_bytes.argtypes = [_vp, C.POINTER(_sz)]
lib.augtree_plan_metadata.argtypes = [_vp, C.c_int, _vp, C.POINTER(_sz)]
lib.augtree_prefill_fwd.argtypes = [_vp] + [_vp] * 5 + [_vp, _sz, _vp]
lib.augtree_replay_fwd.argtypes = [_vp] + [_vp] * 7 + [_vp, _sz, _vp]
lib.augtree_replay_fwd_static.argtypes = [_vp] + [_vp] * 7 + [_vp]
lib.augtree_replay_bwd.argtypes = [_vp] + [_vp] * 13 + [_vp, _sz, _vp]
lib.augtree_prefill_bwd.argtypes = [_vp] + [_vp] * 11 + [_vp, _sz, _vp]
lib.augtree_replay_fwd_state.argtypes = [_vp] + [_vp] * 7 + [C.c_int, _vp, _sz, _vp]
lib.augtree_merge_states.argtypes = [_vp, C.c_int, C.POINTER(_vp), C.POINTER(_vp), _vp, _vp, _vp]
lib.augtree_replay_bwd_state.argtypes = [_vp] + [_vp] * 13 + [C.c_int, _vp, _sz, _vp]
lib.augtree_last_device_status.argtypes = [_vp, C.POINTER(C.c_int), C.POINTER(C.c_int)]
lib.augtree_set_timing.argtypes = [_vp, C.c_int]
lib.augtree_get_kernel_time.argtypes = [_vp, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_int)]
lib.augtree_items_completed.argtypes = [_vp, C.c_int, C.POINTER(C.c_longlong), C.POINTER(C.c_longlong)]
lib.augtree_launch_count.restype = C.c_longlong
lib.augtree_status_string.restype = C.c_char_p
lib.augtree_status_string.argtypes = [C.c_int]


lib.augtree_assign_grid.argtypes = [_i64p, _i64p, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int, _i32p, _i32p, _i64p, _i32p]


PROFILE_FIELDS = ["alpha_p", "beta_p", "lat_p0", "lat_p1", "alpha_tmkv", "beta_tmkv", "lat_tmkv0", "lat_tmkv1", "alpha_mq", "beta_q",
                  "red0", "red1", "lat_mq0", "lat_mq1", "alpha_ring", "beta_ring", "lat_ring0", "lat_ring1", "gamma_ring",
                  "gamma_tmkv", "gamma_mq", "mem_cap", "mem_prompt", "mem_resp"]
RING_CP, TREE_MOVE_KV, MOVE_Q = 0, 1, 2


class ProfileC(C.Structure):
    _fields_ = [(n, C.c_double) for n in PROFILE_FIELDS]


class TreeC(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("prompt_len", C.c_int32), ("n_branches", C.c_int32), ("branch_len", _i32p),
                ("h_q", C.c_int32), ("h_kv", C.c_int32), ("n_degrees", C.c_int32), ("degrees", _i32p), ("b_max", C.c_int32),
                ("exact_max_units", C.c_int32)]


class ChoiceC(C.Structure):
    _fields_ = [("cost", C.c_double), ("degree", C.c_int32), ("primitive", C.c_int32), ("rounds", C.c_int32),
                ("lanes", C.c_int32), ("solved_exactly", C.c_int32), ("n_candidates", C.c_int32)]


lib.augtree_plan_tree.argtypes = [C.POINTER(TreeC), C.POINTER(ProfileC), C.POINTER(ChoiceC), _i32p, _i32p]


def plan_tree(prompt_len, branch_len, h_q, h_kv, degrees, profile: dict, b_max=0, exact_max_units=0):
    """augtree_plan_tree: returns a dict with cost, degree, primitive, rounds, lanes, solved_exactly, n_candidates and the
    placement X as (round[k], lane[k]).  `profile` maps the names in PROFILE_FIELDS to floats (missing: 0)."""
    G = len(branch_len)
    bl = (C.c_int32 * max(G, 1))(*[int(x) for x in branch_len])
    dg = (C.c_int32 * len(degrees))(*[int(x) for x in degrees])
    tree = TreeC(C.sizeof(TreeC), int(prompt_len), G, bl, h_q, h_kv, len(degrees), dg, b_max, exact_max_units)
    prof = ProfileC(*[float(profile.get(n, 0.0)) for n in PROFILE_FIELDS])
    ch = ChoiceC()
    rounds, lanes = (C.c_int32 * max(G, 1))(), (C.c_int32 * max(G, 1))()
    _check(lib.augtree_plan_tree(C.byref(tree), C.byref(prof), C.byref(ch), rounds, lanes), "augtree_plan_tree")
    return {"cost": ch.cost, "degree": ch.degree, "primitive": ch.primitive, "rounds": ch.rounds, "lanes": ch.lanes,
            "solved_exactly": bool(ch.solved_exactly), "n_candidates": ch.n_candidates, "X": (list(rounds[:G]), list(lanes[:G]))}


class AugtreeError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib.augtree_status_string(code).decode()} ({code})")


def _check(code, where):
    if code != 0:
        raise AugtreeError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def assign_grid(weight, size=None, n_rounds=1, n_lanes=1, cell_cap=0, exact_max_units=0):
    """augtree_assign_grid: returns (round[k], lane[k], critical path, solved exactly)."""
    n = len(weight)
    w = (C.c_int64 * max(n, 1))(*[int(x) for x in weight])
    m = None if size is None else (C.c_int64 * max(n, 1))(*[int(x) for x in size])
    rounds, lanes = (C.c_int32 * max(n, 1))(), (C.c_int32 * max(n, 1))()
    path, exact = C.c_int64(0), C.c_int32(0)
    _check(lib.augtree_assign_grid(w, m, n, n_rounds, n_lanes, int(cell_cap), exact_max_units, rounds, lanes,
                                   C.byref(path), C.byref(exact)), "augtree_assign_grid")
    return list(rounds[:n]), list(lanes[:n]), int(path.value), bool(exact.value)


def launch_count() -> int:
    return int(lib.augtree_launch_count())


HANDOFF_LIMIT_BYTES = 0   # default ceiling on the backward hand-off scratch: 0 = recomputing path


class Plan:
    """Owns an augtree_plan_t.  device=None builds a host-only plan (metadata queries only)."""

    def __init__(self, prompt_len, branch_len, h_q, h_kv, head_dim, *, device=0, softmax_scale=0.0, flags=0,
                 n_lanes=0, kv_splits=0):
        self.prompt_len = [int(x) for x in prompt_len]
        self.branch_len = [[int(x) for x in b] for b in branch_len]
        self.h_q, self.h_kv, self.head_dim = h_q, h_kv, head_dim
        self.softmax_scale, self.flags, self.n_lanes, self.kv_splits = softmax_scale, flags, n_lanes, kv_splits
        self.total_p = sum(self.prompt_len)
        self.total_r = sum(sum(b) for b in self.branch_len)
        n = len(self.prompt_len)
        flat = [r for b in self.branch_len for r in b]
        self._pl = (C.c_int32 * n)(*self.prompt_len)
        self._nb = (C.c_int32 * n)(*[len(b) for b in self.branch_len])
        self._bl = (C.c_int32 * max(len(flat), 1))(*flat)
        d = Desc(C.sizeof(Desc), 1, n, self._pl, self._nb, self._bl, h_q, h_kv, head_dim, softmax_scale, flags,
                 n_lanes, kv_splits)
        self._h = C.c_void_p()
        self.device = device
        _check(lib.augtree_plan_create(C.byref(d), -1 if device is None else int(device), C.byref(self._h)), "plan_create")
        f, b = _sz(), _sz()
        _check(lib.augtree_plan_workspace_bytes(self._h, C.byref(f), C.byref(b)), "workspace_bytes")
        self.ws_fwd_bytes, self.ws_bwd_bytes = f.value, b.value
        _check(lib.augtree_plan_bwd_handoff_bytes(self._h, C.byref(b)), "bwd_handoff_bytes")
        self.ws_bwd_handoff_bytes = b.value

    def workspace_bytes(self, handoff_limit=HANDOFF_LIMIT_BYTES) -> int:
        """Scratch for all four calls.  The backward calls take the dS hand-off path (five GEMMs per tile pair instead
        of seven) when its scratch fits under `handoff_limit` bytes, else the recomputing path."""
        need = max(self.ws_fwd_bytes, self.ws_bwd_bytes, 256)
        return max(need, self.ws_bwd_handoff_bytes) if self.ws_bwd_handoff_bytes <= handoff_limit else need

    def __del__(self):
        h = getattr(self, "_h", None)
        if h is not None and h.value and lib is not None:
            lib.augtree_plan_destroy(h)
            self._h = None

    def metadata(self, table_id) -> np.ndarray:
        n = _sz()
        _check(lib.augtree_plan_metadata(self._h, table_id, None, C.byref(n)), "plan_metadata")
        out = np.zeros(n.value // 4, dtype=np.int32)
        _check(lib.augtree_plan_metadata(self._h, table_id, out.ctypes.data_as(C.c_void_p), C.byref(n)), "plan_metadata")
        return out

    @staticmethod
    def _stream():
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def prefill_fwd(self, q_p, k_p, v_p, o_p, lse_p, ws=None):
        _check(lib.augtree_prefill_fwd(self._h, _ptr(q_p), _ptr(k_p), _ptr(v_p), _ptr(o_p), _ptr(lse_p), _ptr(ws),
                                       0 if ws is None else ws.numel() * ws.element_size(), self._stream()), "prefill_fwd")

    def replay_fwd(self, q_r, k_r, v_r, k_p, v_p, o_r, lse_r, ws=None):
        _check(lib.augtree_replay_fwd(self._h, _ptr(q_r), _ptr(k_r), _ptr(v_r), _ptr(k_p), _ptr(v_p), _ptr(o_r),
                                      _ptr(lse_r), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                      self._stream()), "replay_fwd")

    def replay_fwd_static(self, q_r, k_r, v_r, k_p, v_p, o_r, lse_r):
        """replay_fwd with the shard scratch taken from the library's built-in 32 MiB device array:
        for callers that cannot allocate a workspace.  Calls on one device share that array."""
        _check(lib.augtree_replay_fwd_static(self._h, _ptr(q_r), _ptr(k_r), _ptr(v_r), _ptr(k_p), _ptr(v_p), _ptr(o_r),
                                             _ptr(lse_r), self._stream()), "replay_fwd_static")

    def replay_fwd_state(self, q_r, k_r, v_r, k_p, v_p, state_o, state_lse, include_own, ws):
        """Partial softmax state of every response query over this plan's prompt keys (+ its own causal prefix)."""
        _check(lib.augtree_replay_fwd_state(self._h, _ptr(q_r), _ptr(k_r), _ptr(v_r), _ptr(k_p), _ptr(v_p), _ptr(state_o),
                                            _ptr(state_lse), int(bool(include_own)), _ptr(ws), ws.numel() * ws.element_size(),
                                            self._stream()), "replay_fwd_state")

    def merge_states(self, states_o, states_lse, o_r, lse_r):
        n = len(states_o)
        po = (C.c_void_p * n)(*[t.data_ptr() for t in states_o])
        pl = (C.c_void_p * n)(*[t.data_ptr() for t in states_lse])
        _check(lib.augtree_merge_states(self._h, n, po, pl, _ptr(o_r), _ptr(lse_r), self._stream()), "merge_states")

    def replay_bwd_state(self, q_r, k_r, v_r, k_p, v_p, o_r, lse_r, do_r, dq_part, dk_r, dv_r, dkp_acc, dvp_acc, include_own, ws):
        _check(lib.augtree_replay_bwd_state(self._h, _ptr(q_r), _ptr(k_r), _ptr(v_r), _ptr(k_p), _ptr(v_p), _ptr(o_r), _ptr(lse_r),
                                            _ptr(do_r), _ptr(dq_part), _ptr(dk_r), _ptr(dv_r), _ptr(dkp_acc), _ptr(dvp_acc),
                                            int(bool(include_own)), _ptr(ws), ws.numel() * ws.element_size(), self._stream()),
               "replay_bwd_state")

    def replay_bwd(self, q_r, k_r, v_r, k_p, v_p, o_r, lse_r, do_r, dq_r, dk_r, dv_r, dkp_acc, dvp_acc, ws):
        _check(lib.augtree_replay_bwd(self._h, _ptr(q_r), _ptr(k_r), _ptr(v_r), _ptr(k_p), _ptr(v_p), _ptr(o_r),
                                      _ptr(lse_r), _ptr(do_r), _ptr(dq_r), _ptr(dk_r), _ptr(dv_r), _ptr(dkp_acc),
                                      _ptr(dvp_acc), _ptr(ws), ws.numel() * ws.element_size(), self._stream()), "replay_bwd")

    def prefill_bwd(self, q_p, k_p, v_p, o_p, lse_p, do_p, dkp_acc, dvp_acc, dq_p, dk_p=None, dv_p=None, ws=None):
        _check(lib.augtree_prefill_bwd(self._h, _ptr(q_p), _ptr(k_p), _ptr(v_p), _ptr(o_p), _ptr(lse_p), _ptr(do_p),
                                       _ptr(dkp_acc), _ptr(dvp_acc), _ptr(dq_p), _ptr(dk_p), _ptr(dv_p), _ptr(ws),
                                       0 if ws is None else ws.numel() * ws.element_size(), self._stream()), "prefill_bwd")

    def set_timing(self, enable: bool):
        _check(lib.augtree_set_timing(self._h, int(enable)), "set_timing")

    def kernel_time(self, kernel: int):
        ms, n = C.c_float(), C.c_int()
        _check(lib.augtree_get_kernel_time(self._h, kernel, C.byref(ms), C.byref(n)), "get_kernel_time")
        return ms.value, n.value

    def items_completed(self, kernel: int):
        """(items the kernel of schedule `kernel` has finished, items handed to its launches) over the plan's lifetime."""
        done, want = C.c_longlong(), C.c_longlong()
        _check(lib.augtree_items_completed(self._h, kernel, C.byref(done), C.byref(want)), "items_completed")
        return done.value, want.value

    def device_status(self):
        s, d = C.c_int(), C.c_int()
        _check(lib.augtree_last_device_status(self._h, C.byref(s), C.byref(d)), "last_device_status")
        return s.value, d.value


def alloc_outputs(plan: Plan, device="cuda", handoff_limit=HANDOFF_LIMIT_BYTES):
    """Device buffers for one forward + backward pass (allocation only)."""
    hq, hkv, d = plan.h_q, plan.h_kv, plan.head_dim
    bf, f32 = torch.bfloat16, torch.float32
    e = lambda *s, dt=bf: torch.empty(s, device=device, dtype=dt)
    tp, tr = plan.total_p, plan.total_r
    return {
        "o_p": e(tp, hq, d), "lse_p": e(hq, tp, dt=f32), "o_r": e(tr, hq, d), "lse_r": e(hq, tr, dt=f32),
        "dq_p": e(tp, hq, d), "dq_r": e(tr, hq, d), "dk_r": e(tr, hkv, d), "dv_r": e(tr, hkv, d),
        "dk_p": torch.zeros((tp, hkv, d), device=device, dtype=f32), "dv_p": torch.zeros((tp, hkv, d), device=device, dtype=f32),
        "ws": torch.empty(plan.workspace_bytes(handoff_limit), device=device, dtype=torch.uint8),
    }


def run_forward_backward(plan: Plan, t, out):
    """The whole hot path, in call order, on the current stream: 4 entry points."""
    plan.prefill_fwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], out["ws"])
    plan.replay_fwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], out["ws"])
    plan.replay_bwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], t["do_r"],
                    out["dq_r"], out["dk_r"], out["dv_r"], out["dk_p"], out["dv_p"], out["ws"])
    plan.prefill_bwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], t["do_p"], out["dk_p"], out["dv_p"],
                     out["dq_p"], None, None, out["ws"])


class HostStep:
    """The whole hot path for callers whose tensors live in (pinned) host memory: every input is copied to the device
    and every result back, with the copies overlapped with the kernels as far as the data flow allows.  Three streams:
    one for the host->device copies in the order the calls need them, the caller's current stream for the entry points
    (each waits only for its own inputs), one for the device->host copies (each result leaves as soon as its call has
    finished).  The caller's stream has joined both copy streams when `run` returns (asynchronously, like the entry
    points).  Copies, waits and slicing only: no arithmetic here.

    chunks = 1: the four calls of the plan, inputs in the order (prompt inputs, response inputs, dO_R, dO_P).
    chunks = K > 1: the response branches are cut, in packed order, into K runs of about equal length, each with a plan
    of its own over the same prompts, and the replay calls run run by run: forward and backward of a run start as soon as
    ITS slices have arrived, and its results leave while the next run computes.  The prompt-KV gradient accumulators take
    one addition per run (Eq. 2's sum, associated differently from the single call: the same values to fp32 rounding);
    everything else is bit for bit the single call's.  The prefill backward runs BEFORE the replay runs here (its share
    of the accumulators is a term of the same sum, and no bf16 copy of them is asked for), so dQ_P leaves early."""

    IN_ORDER = (("q_p", "k_p", "v_p"), ("q_r", "k_r", "v_r"), ("do_r",), ("do_p",))
    OUT_ORDER = (("o_p", "lse_p"), ("o_r", "lse_r"), ("dq_r", "dk_r", "dv_r"), ("dq_p", "dk_p", "dv_p"))

    def __init__(self, plan: Plan, dev_in, dev_out, chunks=1):
        self.plan, self.t, self.out = plan, dev_in, dev_out
        self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
        self.ev_in = [torch.cuda.Event() for _ in self.IN_ORDER]
        self.ev_done = [torch.cuda.Event() for _ in self.OUT_ORDER]
        self.ev_start, self.ev_in_end, self.ev_out_end = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
        self.runs = self._make_runs(chunks) if chunks > 1 and plan.total_r > 0 else []

    def _make_runs(self, chunks):
        """Cut the packed branches into runs; per run: its plan, the row ranges of its responses and of its groups' prompts."""
        plan = self.plan
        branches = [(g, r) for g, rs in enumerate(plan.branch_len) for r in rs]
        chunks = min(chunks, len(branches))
        target, runs, b0, r0, acc = plan.total_r / chunks, [], 0, 0, 0
        cu_p = [0]
        for P in plan.prompt_len:
            cu_p.append(cu_p[-1] + P)
        for b, (g, r) in enumerate(branches):
            acc += r
            if acc >= target * (len(runs) + 1) - 1e-9 or b == len(branches) - 1:
                g0, g1 = branches[b0][0], g
                bl = [[] for _ in range(g0, g1 + 1)]
                for gg, rr in branches[b0:b + 1]:
                    bl[gg - g0].append(rr)
                sub = Plan(plan.prompt_len[g0:g1 + 1], bl, plan.h_q, plan.h_kv, plan.head_dim, device=plan.device,
                           softmax_scale=plan.softmax_scale, flags=plan.flags & ~FLAG_ZERO_PROMPT_GRAD, n_lanes=plan.n_lanes,
                           kv_splits=plan.kv_splits)
                if max(sub.ws_fwd_bytes, sub.ws_bwd_bytes) > self.out["ws"].numel():
                    raise ValueError("workspace of the whole plan is smaller than a run's")
                runs.append({"plan": sub, "r": (r0, acc), "p": (cu_p[g0], cu_p[g1 + 1]),
                             "lse": torch.empty((plan.h_q, acc - r0), device=self.out["lse_r"].device, dtype=torch.float32),
                             "ev_f_in": torch.cuda.Event(), "ev_b_in": torch.cuda.Event(),
                             "ev_f_done": torch.cuda.Event(), "ev_b_done": torch.cuda.Event()})
                b0, r0 = b + 1, acc
        return runs

    def run(self, host_in, host_out):
        if self.runs:
            return self._run_chunked(host_in, host_out)
        plan, t, out = self.plan, self.t, self.out
        main = torch.cuda.current_stream()
        self.ev_start.record(main)                      # the device buffers are free once earlier work on `main` is done
        self.s_in.wait_event(self.ev_start)
        self.s_out.wait_event(self.ev_start)
        with torch.cuda.stream(self.s_in):
            for names, ev in zip(self.IN_ORDER, self.ev_in):
                for k in names:
                    t[k].copy_(host_in[k], non_blocking=True)
                ev.record(self.s_in)
            self.ev_in_end.record(self.s_in)
        calls = (
            lambda: plan.prefill_fwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], out["ws"]),
            lambda: plan.replay_fwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], out["ws"]),
            lambda: plan.replay_bwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], t["do_r"],
                                    out["dq_r"], out["dk_r"], out["dv_r"], out["dk_p"], out["dv_p"], out["ws"]),
            lambda: plan.prefill_bwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], t["do_p"], out["dk_p"], out["dv_p"],
                                     out["dq_p"], None, None, out["ws"]),
        )
        for i, call in enumerate(calls):
            main.wait_event(self.ev_in[i])
            call()
            self.ev_done[i].record(main)
        with torch.cuda.stream(self.s_out):
            for names, ev in zip(self.OUT_ORDER, self.ev_done):
                self.s_out.wait_event(ev)
                for k in names:
                    host_out[k].copy_(out[k], non_blocking=True)
            self.ev_out_end.record(self.s_out)
        main.wait_event(self.ev_in_end)
        main.wait_event(self.ev_out_end)

    def _run_chunked(self, host_in, host_out):
        plan, t, out, runs = self.plan, self.t, self.out, self.runs
        main = torch.cuda.current_stream()
        self.ev_start.record(main)
        self.s_in.wait_event(self.ev_start)
        self.s_out.wait_event(self.ev_start)
        # ---- host -> device, in the order the calls can use them: the prompt's inputs and dO_P, then per run its q/k/v and dO
        with torch.cuda.stream(self.s_in):
            for k in ("q_p", "k_p", "v_p"):
                t[k].copy_(host_in[k], non_blocking=True)
            self.ev_in[0].record(self.s_in)
            t["do_p"].copy_(host_in["do_p"], non_blocking=True)
            self.ev_in[3].record(self.s_in)
            for run in runs:
                a, b = run["r"]
                for k in ("q_r", "k_r", "v_r"):
                    t[k][a:b].copy_(host_in[k][a:b], non_blocking=True)
                run["ev_f_in"].record(self.s_in)
                t["do_r"][a:b].copy_(host_in["do_r"][a:b], non_blocking=True)
                run["ev_b_in"].record(self.s_in)
            self.ev_in_end.record(self.s_in)
        # ---- the calls.  The prompt-KV accumulators are sums (Eq. 2 plus the prefill's own part): with no bf16 copy of
        # them asked for, the prefill backward may add its part first, so that dQ_P leaves while the replay runs compute.
        if plan.flags & FLAG_ZERO_PROMPT_GRAD:      # the runs' plans do not clear: each ADDS its share of Eq. 2's sum
            out["dk_p"].zero_()
            out["dv_p"].zero_()
        main.wait_event(self.ev_in[0])
        plan.prefill_fwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], out["ws"])
        self.ev_done[0].record(main)
        main.wait_event(self.ev_in[3])
        plan.prefill_bwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], t["do_p"], out["dk_p"], out["dv_p"], out["dq_p"],
                         None, None, out["ws"])      # (adds its share; it never clears the accumulators)
        self.ev_done[3].record(main)
        for run in runs:
            sub, (a, b), (pa, pb) = run["plan"], run["r"], run["p"]
            kp, vp = t["k_p"][pa:pb], t["v_p"][pa:pb]
            main.wait_event(run["ev_f_in"])
            sub.replay_fwd(t["q_r"][a:b], t["k_r"][a:b], t["v_r"][a:b], kp, vp, out["o_r"][a:b], run["lse"], out["ws"])
            out["lse_r"][:, a:b].copy_(run["lse"], non_blocking=True)     # LSE is head-major: a run's columns are strided
            run["ev_f_done"].record(main)
            main.wait_event(run["ev_b_in"])
            sub.replay_bwd(t["q_r"][a:b], t["k_r"][a:b], t["v_r"][a:b], kp, vp, out["o_r"][a:b], run["lse"], t["do_r"][a:b],
                           out["dq_r"][a:b], out["dk_r"][a:b], out["dv_r"][a:b], out["dk_p"][pa:pb], out["dv_p"][pa:pb], out["ws"])
            run["ev_b_done"].record(main)
        # ---- device -> host, each result as soon as its call is done
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_done[0])
            for k in ("o_p", "lse_p"):
                host_out[k].copy_(out[k], non_blocking=True)
            self.s_out.wait_event(self.ev_done[3])
            host_out["dq_p"].copy_(out["dq_p"], non_blocking=True)
            for run in runs:
                a, b = run["r"]
                self.s_out.wait_event(run["ev_f_done"])
                host_out["o_r"][a:b].copy_(out["o_r"][a:b], non_blocking=True)
                self.s_out.wait_event(run["ev_b_done"])
                for k in ("dq_r", "dk_r", "dv_r"):
                    host_out[k][a:b].copy_(out[k][a:b], non_blocking=True)
            for k in ("lse_r", "dk_p", "dv_p"):
                host_out[k].copy_(out[k], non_blocking=True)
            self.ev_out_end.record(self.s_out)
        main.wait_event(self.ev_in_end)
        main.wait_event(self.ev_out_end)


def capture_step(plan: Plan, t, out):
    """The whole hot path captured once into a CUDA graph (the library allocates nothing and does not synchronise
    in its launch path); `graph.replay()` then re-runs it on the same buffers.  Pays off for launch-bound sizes."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        run_forward_backward(plan, t, out)  # first use of each kernel sets its attributes: keep that out of the capture
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            run_forward_backward(plan, t, out)
    torch.cuda.current_stream().wait_stream(s)
    return g
