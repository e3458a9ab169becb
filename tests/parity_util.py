"""Shared helpers of the GPU parity tests: run the CUDA path and the fp64 oracle on the same inputs.

Tolerances (the benchmark contract's, against fp64): per tensor, relative L2 error <= 5e-3 and largest
absolute error <= 2e-2 for O and the six gradients; |LSE error| <= 1e-3.  `assert_parity` asserts exactly
these.  Two things are allowed to differ, and only where a test says so by name:

* `exceptions` widens one bound of one tensor for one named test case, with the measured value in the test.
* `assert_parity_elementwise` replaces the flat absolute bound, element by element, by
  max(2e-2, six standard deviations of that element's modelled rounding error), for the random sweep and for
  gradients handed back in bf16.  The relative-L2 bound stays as stated.
"""
import numpy as np
import torch

from oracle import tree_attention as ora
from paper_2609_33133_b200 import workloads as wl

REL_L2, MAX_ABS, LSE_ABS = 5e-3, 2e-2, 1e-3   # tolerances of the benchmark contract, against fp64
GRADS = ["dq_p", "dk_p", "dv_p", "dq_r", "dk_r", "dv_r"]
U_BF16 = 2.0 ** -8                            # unit roundoff of bf16, round to nearest (8 significant bits)


def run_gpu(B, w, t_cpu, kv_splits=0, n_lanes=0, flags=0, handoff_limit=None):
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0, kv_splits=kv_splits,
                  n_lanes=n_lanes, flags=flags)
    t = {k: v.cuda() for k, v in t_cpu.items()}
    out = B.alloc_outputs(plan) if handoff_limit is None else B.alloc_outputs(plan, handoff_limit=handoff_limit)
    B.run_forward_backward(plan, t, out)
    torch.cuda.synchronize()
    status = plan.device_status()
    assert status == (0, 0), f"device status {status}"
    return {k: v.float().cpu().numpy().astype(np.float64) for k, v in out.items() if k != "ws"}, plan


def run_oracle(w, t_cpu):
    tb = ora.TreeBatch(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim)
    f = lambda x: x.float().numpy().astype(np.float64)
    return ora.tree_attention_fwd_bwd(tb, *[f(t_cpu[n]) for n in wl.TENSOR_NAMES])


def errors(got, ref):
    rows = {}
    for k in ref:
        if ref[k].size == 0:
            continue
        diff = got[k] - ref[k]
        finite = np.isfinite(got[k]).all()
        denom = np.linalg.norm(ref[k].ravel())
        rows[k] = (float(np.linalg.norm(diff.ravel()) / denom) if denom > 0 else 0.0, float(np.abs(diff).max()), bool(finite))
    return rows


def assert_parity(got, ref, exceptions=None):
    """The stated tolerances on every tensor.  `exceptions`: {tensor: {"max_abs": x} or {"rel_l2": x}} for a
    named case whose test states the measured value and why."""
    rows = errors(got, ref)
    exceptions = exceptions or {}
    bad = []
    for k, (rel, mx, finite) in rows.items():
        ex = exceptions.get(k, {})
        if not finite:
            bad.append((k, "non-finite"))
        elif k.startswith("lse"):
            if mx > LSE_ABS:
                bad.append((k, rel, mx))
        elif rel > ex.get("rel_l2", REL_L2) or mx > ex.get("max_abs", MAX_ABS):
            bad.append((k, rel, mx, float(np.abs(ref[k]).max())))
    assert not bad, f"parity failures: {bad}; all: {rows}"
    return rows


# --------------------------------------------------------------------------- #
# First-order model of the kernels' rounding error, element by element.
#
# The kernels keep every accumulation in fp32 and round to bf16 in exactly these places: P before the P V and
# P^T dO products, dS before the dS K and dS^T Q products, O on delivery (delta = rowsum(dO * O) is taken from
# that delivered O), and the bf16-delivered gradients on delivery.  Round-to-nearest to 8 significant bits
# leaves an error uniform in +-half an ulp: zero mean, |error| <= u |x| with unit roundoff u = 2^-8, standard
# deviation <= u |x| / sqrt(3).  The roundings are independent, so to first order, with p, dS, delta the exact
# quantities of one (sequence, head) and r = u^2 / 3:
#   var O_ad     = r (sum_b p_ab^2 V_bd^2 + O_ad^2)                                  (P rounded; delivery)
#   var delta_a  = sum_d dO_ad^2 var O_ad
#   var dQ_ad    = scale^2 (r sum_b dS_ab^2 K_bd^2 + var delta_a (sum_b p_ab K_bd)^2)   [+ r dQ_ad^2 on delivery]
#   var dK_bd    = scale^2 sum_a (r dS_ab^2 + p_ab^2 var delta_a) Q_ad^2                 [+ r dK_bd^2 on delivery]
#   var dV_bd    = r sum_a p_ab^2 dO_ad^2                                             [+ r dV_bd^2 on delivery]
# (the error of delta_a is common to the whole row a, so it enters dQ_a coherently; fp32 accumulation and the
# exp2 approximations are two to four orders of magnitude below u and are left out), and variances add over
# the query heads and branches that are summed into one element.  Over the many keys of an ordinary row the
# standard deviation is a few 1e-4.  It is large only where a row's softmax sits on a handful of keys (the
# first rows of a sequence, rows right behind a one- or two-token prompt): there p ~ 1, dS = p (dP - delta) is
# of order sqrt(d) ~ 10, and one bf16 rounding of it is up to 4e-2 before it is multiplied by scale * K.
# The element-wise bound asserted is max(2e-2, SIGMAS x standard deviation).
SIGMAS = 6.0


def rounding_error_sigma(w, t_cpu, bf16_prompt_grads=False):
    """Standard deviation of the modelled rounding error of every element of o_*, d*_p, d*_r."""
    tb = ora.TreeBatch(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim)
    f = lambda x: x.float().numpy().astype(np.float64)
    q_p, k_p, v_p, do_p, q_r, k_r, v_r, do_r = [f(t_cpu[n]) for n in wl.TENSOR_NAMES]
    hq, hkv, scale = tb.h_q, tb.h_kv, tb.scale
    r = U_BF16 ** 2 / 3.0
    rep = hq // hkv
    var = {"o_p": np.zeros_like(q_p), "o_r": np.zeros_like(q_r), "dq_p": np.zeros_like(q_p), "dk_p": np.zeros_like(k_p),
           "dv_p": np.zeros_like(v_p), "dq_r": np.zeros_like(q_r), "dk_r": np.zeros_like(k_r), "dv_r": np.zeros_like(v_r)}
    exact = {k: np.zeros_like(v) for k, v in var.items()}   # the exact values, for the delivery-rounding terms
    for g in range(tb.n_groups):
        p0, p1 = int(tb.cu_p[g]), int(tb.cu_p[g + 1])
        P = p1 - p0
        G = len(tb.branch_len[g])
        branches = [(0, 0)] if G == 0 else [(int(tb.cu_r[tb.cu_b[g] + i]), int(tb.cu_r[tb.cu_b[g] + i + 1])) for i in range(G)]
        for h in range(hq):
            c = h // rep
            for n_copy, (r0, r1) in enumerate(branches):
                q = np.concatenate([q_p[p0:p1, h], q_r[r0:r1, h]])
                k = np.concatenate([k_p[p0:p1, c], k_r[r0:r1, c]])
                v = np.concatenate([v_p[p0:p1, c], v_r[r0:r1, c]])
                # the kernels run the prompt rows once, under the whole seed dO_P: the copy that carries them here
                # is the first one; the other copies contribute their response rows only
                do = np.concatenate([do_p[p0:p1, h] if n_copy == 0 else np.zeros((P, q.shape[1])), do_r[r0:r1, h]])
                o, _, p = ora.causal_attention_fwd(q, k, v, scale)
                dq, dk, dv = ora.causal_attention_bwd(q, k, v, o, p, do, scale)
                var_o = r * ((p * p) @ (v * v) + o * o)
                var_delta = ((do * do) * var_o).sum(axis=1, keepdims=True)
                ds = p * (do @ v.T - (do * o).sum(axis=1, keepdims=True))
                v_dq = scale ** 2 * (r * ((ds * ds) @ (k * k)) + var_delta * (p @ k) ** 2)
                v_dk = scale ** 2 * ((r * ds * ds + p * p * var_delta).T @ (q * q))
                v_dv = r * ((p * p).T @ (do * do))
                if n_copy == 0:
                    var["o_p"][p0:p1, h] = var_o[:P]
                var["o_r"][r0:r1, h] = var_o[P:]
                for name, vv, ex, hd in (("dq", v_dq, dq, h), ("dk", v_dk, dk, c), ("dv", v_dv, dv, c)):
                    var[name + "_p"][p0:p1, hd] += vv[:P]; exact[name + "_p"][p0:p1, hd] += ex[:P]
                    var[name + "_r"][r0:r1, hd] += vv[P:]; exact[name + "_r"][r0:r1, hd] += ex[P:]
    delivered_bf16 = ["dq_p", "dq_r", "dk_r", "dv_r"] + (["dk_p", "dv_p"] if bf16_prompt_grads else [])
    for name in delivered_bf16:
        var[name] += r * exact[name] ** 2
    return {name: np.sqrt(x) for name, x in var.items()}


def assert_parity_elementwise(got, ref, sigma, rel_l2=None):
    """rel-L2 <= 5e-3 per tensor and |LSE error| <= 1e-3 as stated; the absolute error of every element
    <= max(2e-2, SIGMAS x its modelled rounding-error standard deviation).  `rel_l2`: {tensor: bound} for a
    named case whose test states why."""
    rel_l2 = rel_l2 or {}
    rows = errors(got, ref)
    bad = []
    for k, (rel, mx, finite) in rows.items():
        if not finite:
            bad.append((k, "non-finite"))
        elif k.startswith("lse"):
            if mx > LSE_ABS:
                bad.append((k, rel, mx))
        else:
            bound = np.maximum(MAX_ABS, SIGMAS * sigma[k])
            over = np.abs(got[k] - ref[k]) - bound
            if rel > rel_l2.get(k, REL_L2) or over.max() > 0:
                i = np.unravel_index(int(np.argmax(over)), over.shape)
                bad.append((k, rel, mx, "worst element", i, float(np.abs(got[k] - ref[k])[i]), "bound", float(bound[i])))
    assert not bad, f"parity failures: {bad}; all: {rows}"
    return rows


class SampledError:
    """The stated tolerances on a sample of rows of one full-size tensor: every sampled element within the
    absolute bound, and the relative L2 error over the whole sample (the sample's estimate of the tensor's
    figure) within 5e-3."""

    def __init__(self, name, max_abs=MAX_ABS):
        self.name, self.max_abs, self.num, self.den, self.worst, self.n = name, max_abs, 0.0, 0.0, 0.0, 0

    def add(self, got, ref, where=None):
        got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
        err = np.abs(got - ref)
        assert np.isfinite(got).all(), (self.name, where)
        assert err.max() <= self.max_abs, (self.name, where, float(err.max()), float(np.abs(ref).max()))
        self.num += float((err ** 2).sum()); self.den += float((ref ** 2).sum()); self.n += 1
        self.worst = max(self.worst, float(err.max()))

    def check(self):
        assert self.n > 0, self.name
        rel = (self.num / self.den) ** 0.5 if self.den > 0 else 0.0
        assert rel <= REL_L2, (self.name, "rel-L2 over the sample", rel)
        return rel, self.worst
