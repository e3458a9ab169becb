"""Plain fp64 oracle for prompt-sharing tree attention, forward and backward.

TEST INFRASTRUCTURE ONLY.  Imported by the tests, by the smoke check and by
the benchmark's CPU-baseline leg; never by the product path.  It shares no
code, constants or helpers with the CUDA kernels.

What it computes (all in float64 on the exact input values):

* The replay tree T = (P, {R_i}, i = 1..G) of Sec. 3.1 is *flattened* into the
  G linear sequences (P, R_i) of Sec. 2.1 ("Replay tree").
* On every flattened sequence, for every query head, ordinary causal
  scaled-dot-product attention  O = softmax(Q K^T / sqrt(D_h) + M) V  of
  Sec. 2.2 ("Attention as block interactions").  The mask lets row a see the
  keys b <= a (inclusive diagonal: the "standard causal mask" of Sec. 3.4;
  Eq. 1 then gives a response token the whole prompt plus its own prefix and
  nothing from sibling branches, because siblings are in other sequences).
* The backward pass is the textbook derivative of that formula, written out
  with explicit n x n matrices.
* Prompt-side results: the prompt rows of every flattened copy produce the
  same O and LSE (asserted), and the prompt gradients are the sum over the G
  copies, which is Eq. 2 plus the prefill graph's own contribution
  (Sec. 3.2, "Exact many-to-one backward").

Layouts (shared with the library's C interface, but restated here):
  q_p, do_p : [sum P, H_q, d]      k_p, v_p : [sum P, H_kv, d]
  q_r, do_r : [sum R, H_q, d]      k_r, v_r : [sum R, H_kv, d]
prompts of the groups back to back; responses group-major, branch order.
LSE is [H_q, tokens], natural log of the scaled scores' sum of exponentials
(LSE = m + ln l in the (m, l, O_acc) notation of Sec. 3.3).
Query head h reads KV head h // (H_q / H_kv).

Parity pins (tests/test_oracle_pins.py): central finite differences, the dense
tree-mask formulation, split + merge of partial softmax states, torch's
scaled_dot_product_attention for G = 1, closed forms (zero keys, constant
values, first row), and row-sum invariants.  Every function below is covered
by at least one of them.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------- #
# One linear causal sequence, one head (Sec. 2.2 definition, written out).
# --------------------------------------------------------------------------- #
def causal_attention_fwd(q, k, v, scale):
    """O, LSE and the probability matrix of causal attention on one sequence.

    q, k, v: [n, d] float64.  Row a attends to keys b <= a.
    Returns (o [n, d], lse [n], p [n, n]).
    """
    n = q.shape[0]
    s = scale * (q @ k.T)
    visible = np.tril(np.ones((n, n), dtype=bool))
    s = np.where(visible, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    p = e / l
    o = p @ v
    lse = (m + np.log(l))[:, 0]
    return o, lse, p


def causal_attention_bwd(q, k, v, o, p, do, scale):
    """Gradients of sum(O * dO) with respect to q, k, v for one sequence.

    With p = softmax(s) row-wise and o = p v:
      dv = p^T do;  dp = do v^T;  ds = p * (dp - rowsum(do * o));
      dq = scale * ds k;  dk = scale * ds^T q.
    """
    delta = (do * o).sum(axis=1, keepdims=True)
    dv = p.T @ do
    dp = do @ v.T
    ds = p * (dp - delta)
    dq = scale * (ds @ k)
    dk = scale * (ds.T @ q)
    return dq, dk, dv


# --------------------------------------------------------------------------- #
# Descriptor helpers (pure bookkeeping).
# --------------------------------------------------------------------------- #
class TreeBatch:
    """Lengths of a batch of replay trees: prompt_len[g], branch_len[g][i]."""

    def __init__(self, prompt_len, branch_len, h_q, h_kv, head_dim, scale=None):
        self.prompt_len = [int(x) for x in prompt_len]
        self.branch_len = [[int(x) for x in b] for b in branch_len]
        assert len(self.prompt_len) == len(self.branch_len)
        self.h_q, self.h_kv, self.head_dim = int(h_q), int(h_kv), int(head_dim)
        assert self.h_q % self.h_kv == 0
        self.scale = float(scale) if scale else 1.0 / np.sqrt(self.head_dim)
        self.cu_p = np.concatenate([[0], np.cumsum(self.prompt_len)]).astype(np.int64)
        flat = [r for b in self.branch_len for r in b]
        self.cu_r = np.concatenate([[0], np.cumsum(flat)]).astype(np.int64)
        self.cu_b = np.concatenate([[0], np.cumsum([len(b) for b in self.branch_len])]).astype(np.int64)

    @property
    def n_groups(self):
        return len(self.prompt_len)


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


# --------------------------------------------------------------------------- #
# The oracle proper: flatten, attend, differentiate, reduce.
# --------------------------------------------------------------------------- #
def tree_attention_fwd_bwd(tb, q_p, k_p, v_p, do_p, q_r, k_r, v_r, do_r, with_backward=True):
    """Forward and backward of tree attention through the flattened definition.

    For group g, branch i, query head h (KV head c = h // (H_q/H_kv)) build the
    linear sequence [prompt; response i], run causal attention, and, for the
    backward, seed the response rows with do_r and the prompt rows of each of
    the G copies with do_p / G (the prompt-row outputs of all copies are the
    same function of the same inputs, so their seeds add up to do_p).

    Returns a dict with o_p, lse_p, o_r, lse_r and, if with_backward,
    dq_p, dk_p, dv_p, dq_r, dk_r, dv_r (all float64, layouts as the inputs;
    dk/dv summed over the query heads that share a KV head; prompt gradients
    summed over the branches, Eq. 2).
    """
    q_p, k_p, v_p, do_p = _f64(q_p), _f64(k_p), _f64(v_p), _f64(do_p)
    q_r, k_r, v_r, do_r = _f64(q_r), _f64(k_r), _f64(v_r), _f64(do_r)
    hq, hkv, scale = tb.h_q, tb.h_kv, tb.scale
    rep = hq // hkv
    out = {
        "o_p": np.zeros_like(q_p), "lse_p": np.zeros((hq, q_p.shape[0])),
        "o_r": np.zeros_like(q_r), "lse_r": np.zeros((hq, q_r.shape[0])),
    }
    if with_backward:
        out.update({
            "dq_p": np.zeros_like(q_p), "dk_p": np.zeros_like(k_p), "dv_p": np.zeros_like(v_p),
            "dq_r": np.zeros_like(q_r), "dk_r": np.zeros_like(k_r), "dv_r": np.zeros_like(v_r),
        })
    for g in range(tb.n_groups):
        p0, p1 = int(tb.cu_p[g]), int(tb.cu_p[g + 1])
        P = p1 - p0
        G = len(tb.branch_len[g])
        if G == 0:
            # A prompt with no responses: the tree is the prompt alone.
            branches = [(None, 0, 0)]
            n_copies = 1
        else:
            branches = [(i, int(tb.cu_r[tb.cu_b[g] + i]), int(tb.cu_r[tb.cu_b[g] + i + 1])) for i in range(G)]
            n_copies = G
        for h in range(hq):
            c = h // rep
            first_o = first_lse = None
            for (i, r0, r1) in branches:
                q = np.concatenate([q_p[p0:p1, h], q_r[r0:r1, h]], axis=0)
                k = np.concatenate([k_p[p0:p1, c], k_r[r0:r1, c]], axis=0)
                v = np.concatenate([v_p[p0:p1, c], v_r[r0:r1, c]], axis=0)
                o, lse, p = causal_attention_fwd(q, k, v, scale)
                if first_o is None:
                    first_o, first_lse = o[:P], lse[:P]
                    out["o_p"][p0:p1, h] = first_o
                    out["lse_p"][h, p0:p1] = first_lse
                else:
                    # every flattened copy recomputes the same prompt rows
                    assert np.allclose(o[:P], first_o, rtol=1e-12, atol=1e-12)
                    assert np.allclose(lse[:P], first_lse, rtol=1e-12, atol=1e-12)
                out["o_r"][r0:r1, h] = o[P:]
                out["lse_r"][h, r0:r1] = lse[P:]
                if not with_backward:
                    continue
                do = np.concatenate([do_p[p0:p1, h] / n_copies, do_r[r0:r1, h]], axis=0)
                dq, dk, dv = causal_attention_bwd(q, k, v, o, p, do, scale)
                out["dq_p"][p0:p1, h] += dq[:P]
                out["dk_p"][p0:p1, c] += dk[:P]
                out["dv_p"][p0:p1, c] += dv[:P]
                out["dq_r"][r0:r1, h] = dq[P:]
                out["dk_r"][r0:r1, c] += dk[P:]
                out["dv_r"][r0:r1, c] += dv[P:]
    return out


# --------------------------------------------------------------------------- #
# Row-at-a-time forms of the same definition, for spot checks at sizes where
# the n x n matrices above do not fit.  Same formulas, one query row.
# --------------------------------------------------------------------------- #
def forward_row(tb, q_p, k_p, v_p, q_r, k_r, v_r, kind, token, head):
    """O row and LSE of one query: kind 'p' (prompt token) or 'r' (response token).

    token indexes the packed prompt or response token axis.  The visible keys
    are the prompt prefix (prompt query) or the whole prompt of the group plus
    the branch prefix up to and including the token itself (Eq. 1).
    """
    hq, hkv = tb.h_q, tb.h_kv
    c = head // (hq // hkv)
    if kind == "p":
        g = int(np.searchsorted(tb.cu_p, token, side="right") - 1)
        p0 = int(tb.cu_p[g])
        q = np.asarray(q_p[token, head], dtype=np.float64)
        k = np.asarray(k_p[p0:token + 1, c], dtype=np.float64)
        v = np.asarray(v_p[p0:token + 1, c], dtype=np.float64)
    else:
        b = int(np.searchsorted(tb.cu_r, token, side="right") - 1)
        g = int(np.searchsorted(tb.cu_b, b, side="right") - 1)
        p0, p1 = int(tb.cu_p[g]), int(tb.cu_p[g + 1])
        r0 = int(tb.cu_r[b])
        q = np.asarray(q_r[token, head], dtype=np.float64)
        k = np.concatenate([np.asarray(k_p[p0:p1, c], dtype=np.float64),
                            np.asarray(k_r[r0:token + 1, c], dtype=np.float64)], axis=0)
        v = np.concatenate([np.asarray(v_p[p0:p1, c], dtype=np.float64),
                            np.asarray(v_r[r0:token + 1, c], dtype=np.float64)], axis=0)
    s = tb.scale * (k @ q)
    m = s.max()
    e = np.exp(s - m)
    l = e.sum()
    return (e / l) @ v, m + np.log(l)


def dq_row(tb, q_p, k_p, v_p, do_p, q_r, k_r, v_r, do_r, kind, token, head):
    """Gradient of one query row (it depends on that row's own softmax only).

    For a prompt query the seeds of the G flattened copies add up to do_p, and
    the row is the same in every copy, so the sum over copies is the gradient
    under the full seed.
    """
    hq, hkv = tb.h_q, tb.h_kv
    c = head // (hq // hkv)
    if kind == "p":
        g = int(np.searchsorted(tb.cu_p, token, side="right") - 1)
        p0 = int(tb.cu_p[g])
        q = np.asarray(q_p[token, head], dtype=np.float64)
        do = np.asarray(do_p[token, head], dtype=np.float64)
        k = np.asarray(k_p[p0:token + 1, c], dtype=np.float64)
        v = np.asarray(v_p[p0:token + 1, c], dtype=np.float64)
    else:
        b = int(np.searchsorted(tb.cu_r, token, side="right") - 1)
        g = int(np.searchsorted(tb.cu_b, b, side="right") - 1)
        p0, p1 = int(tb.cu_p[g]), int(tb.cu_p[g + 1])
        r0 = int(tb.cu_r[b])
        q = np.asarray(q_r[token, head], dtype=np.float64)
        do = np.asarray(do_r[token, head], dtype=np.float64)
        k = np.concatenate([np.asarray(k_p[p0:p1, c], dtype=np.float64),
                            np.asarray(k_r[r0:token + 1, c], dtype=np.float64)], axis=0)
        v = np.concatenate([np.asarray(v_p[p0:p1, c], dtype=np.float64),
                            np.asarray(v_r[r0:token + 1, c], dtype=np.float64)], axis=0)
    s = tb.scale * (k @ q)
    e = np.exp(s - s.max())
    p = e / e.sum()
    o = p @ v
    ds = p * (v @ do - do @ o)
    return tb.scale * (ds @ k)


def dkv_key(tb, q_p, k_p, v_p, do_p, q_r, k_r, v_r, do_r, kind, token, kv_head):
    """dK and dV of one key (kind 'p' prompt / 'r' response, packed token index, KV head).

    Sums, over every query row that sees the key and every query head of the KV
    head, p_ab * dO_a (dV) and scale * dS_ab * q_a (dK), each row's softmax taken
    over that row's full visible key set.  For a prompt key the rows are the later
    prompt rows and every response row of every branch of the group (Eq. 2).
    Cost grows with the number of rows, so use it for keys few rows can see.
    """
    hq, hkv = tb.h_q, tb.h_kv
    rep = hq // hkv
    d = tb.head_dim
    dk, dv = np.zeros(d), np.zeros(d)
    if kind == "p":
        g = int(np.searchsorted(tb.cu_p, token, side="right") - 1)
        rows = [("p", a) for a in range(token, int(tb.cu_p[g + 1]))]
        for b in range(int(tb.cu_b[g]), int(tb.cu_b[g + 1])):
            rows += [("r", a) for a in range(int(tb.cu_r[b]), int(tb.cu_r[b + 1]))]
        kvec = np.asarray(k_p[token, kv_head], dtype=np.float64)
        vvec = np.asarray(v_p[token, kv_head], dtype=np.float64)
    else:
        b = int(np.searchsorted(tb.cu_r, token, side="right") - 1)
        rows = [("r", a) for a in range(token, int(tb.cu_r[b + 1]))]
        kvec = np.asarray(k_r[token, kv_head], dtype=np.float64)
        vvec = np.asarray(v_r[token, kv_head], dtype=np.float64)
    for (rk, a) in rows:
        for h in range(kv_head * rep, (kv_head + 1) * rep):
            o, lse = forward_row(tb, q_p, k_p, v_p, q_r, k_r, v_r, rk, a, h)
            q = np.asarray((q_p if rk == "p" else q_r)[a, h], dtype=np.float64)
            do = np.asarray((do_p if rk == "p" else do_r)[a, h], dtype=np.float64)
            p_ab = np.exp(tb.scale * (q @ kvec) - lse)
            dv += p_ab * do
            ds = p_ab * (do @ vvec - do @ o)
            dk += tb.scale * ds * q
    return dk, dv


def dkv_keys_block(tb, q_p, k_p, v_p, do_p, q_r, k_r, v_r, do_r, kind, tokens, kv_head, block=256):
    """dK and dV of several keys of ONE sequence part (all `tokens` prompt tokens of one group, kind 'p',
    or response tokens of one branch, kind 'r') and one KV head: the sums of dkv_key, taken a block of
    query rows at a time so that each row's softmax over its full visible key set is one matrix product.

    Rows that see a prompt key: the prompt rows from the key on, and every response row of every branch
    of the group (Eq. 2).  Rows that see a response key: the rows of its branch from the key on.
    Returns (dk [len(tokens), d], dv [len(tokens), d]).  Same formulas as dkv_key; pinned against it.
    """
    hq, hkv, scale = tb.h_q, tb.h_kv, tb.scale
    rep = hq // hkv
    tokens = [int(x) for x in tokens]
    f = lambda x: np.asarray(x, dtype=np.float64)
    if kind == "p":
        g = int(np.searchsorted(tb.cu_p, tokens[0], side="right") - 1)
        seq0, seq1 = int(tb.cu_p[g]), int(tb.cu_p[g + 1])
        branches = range(int(tb.cu_b[g]), int(tb.cu_b[g + 1]))
    else:
        b = int(np.searchsorted(tb.cu_r, tokens[0], side="right") - 1)
        g = int(np.searchsorted(tb.cu_b, b, side="right") - 1)
        seq0, seq1 = int(tb.cu_r[b]), int(tb.cu_r[b + 1])
        branches = []
    assert all(seq0 <= t < seq1 for t in tokens), "keys must lie in one prompt / one branch"
    p0, p1 = int(tb.cu_p[g]), int(tb.cu_p[g + 1])
    kp, vp = f(k_p[p0:p1, kv_head]), f(v_p[p0:p1, kv_head])
    key_pos = np.asarray([t - seq0 for t in tokens])           # position inside the key's own sequence part
    dk, dv = np.zeros((len(tokens), tb.head_dim)), np.zeros((len(tokens), tb.head_dim))

    def rows_block(q, do, keys_k, keys_v, first_pos, own_len, sel_cols, sel_visible):
        """q, do: [m, d] rows at positions first_pos.. of a causal range of own_len keys that follows an
        unmasked range; keys_*: [unmasked + own_len, d]; adds the rows' terms for the key columns sel_cols
        (sel_visible[m, n_sel]: whether row sees that key)."""
        m = q.shape[0]
        n_un = keys_k.shape[0] - own_len
        s = scale * (q @ keys_k.T)
        pos = first_pos + np.arange(m)
        col = np.arange(keys_k.shape[0])
        s = np.where(col[None, :] <= n_un + pos[:, None], s, -np.inf)
        mx = s.max(axis=1, keepdims=True)
        e = np.exp(s - mx)
        p = e / e.sum(axis=1, keepdims=True)
        o = p @ keys_v
        delta = (do * o).sum(axis=1)
        inside = sel_cols < keys_k.shape[0]          # a key past the block's last row is in no row's range
        cols = np.where(inside, sel_cols, 0)
        psel = np.where(sel_visible & inside[None, :], p[:, cols], 0.0)             # [m, n_sel]
        dsel = psel * (do @ keys_v[cols].T - delta[:, None])
        return scale * (dsel.T @ q), psel.T @ do

    for h in range(kv_head * rep, (kv_head + 1) * rep):
        if kind == "p":
            # later prompt rows of the same prompt (causal inside the prompt)
            lo = int(key_pos.min())
            for a0 in range(lo, p1 - p0, block):
                a1 = min(a0 + block, p1 - p0)
                vis = (a0 + np.arange(a1 - a0))[:, None] >= key_pos[None, :]
                ddk, ddv = rows_block(f(q_p[p0 + a0:p0 + a1, h]), f(do_p[p0 + a0:p0 + a1, h]), kp[:a1], vp[:a1], a0, a1, key_pos, vis)
                dk += ddk; dv += ddv
            # every response row of every branch of the group (unmasked on the prompt)
            for bi in branches:
                r0, r1 = int(tb.cu_r[bi]), int(tb.cu_r[bi + 1])
                kr, vr = f(k_r[r0:r1, kv_head]), f(v_r[r0:r1, kv_head])
                for a0 in range(0, r1 - r0, block):
                    a1 = min(a0 + block, r1 - r0)
                    kk, vv = np.concatenate([kp, kr[:a1]]), np.concatenate([vp, vr[:a1]])
                    vis = np.ones((a1 - a0, len(tokens)), dtype=bool)
                    ddk, ddv = rows_block(f(q_r[r0 + a0:r0 + a1, h]), f(do_r[r0 + a0:r0 + a1, h]), kk, vv, a0, a1, key_pos, vis)
                    dk += ddk; dv += ddv
        else:
            kr, vr = f(k_r[seq0:seq1, kv_head]), f(v_r[seq0:seq1, kv_head])
            lo = int(key_pos.min())
            for a0 in range(lo, seq1 - seq0, block):
                a1 = min(a0 + block, seq1 - seq0)
                kk, vv = np.concatenate([kp, kr[:a1]]), np.concatenate([vp, vr[:a1]])
                vis = (a0 + np.arange(a1 - a0))[:, None] >= key_pos[None, :]
                ddk, ddv = rows_block(f(q_r[seq0 + a0:seq0 + a1, h]), f(do_r[seq0 + a0:seq0 + a1, h]), kk, vv, a0, a1,
                                      (p1 - p0) + key_pos, vis)
                dk += ddk; dv += ddv
    return dk, dv


# --------------------------------------------------------------------------- #
# Second and third formulations, used only to pin the one above.
# --------------------------------------------------------------------------- #
def tree_mask(P, branch_len):
    """Boolean visibility matrix over the token order [P; R_1; ...; R_G].

    A shared prompt column (causal inside the prompt) plus block-diagonal
    causal response blocks (Sec. 2.2, "Replay mismatch"; Eq. 1).
    """
    n = P + sum(branch_len)
    vis = np.zeros((n, n), dtype=bool)
    vis[:P, :P] = np.tril(np.ones((P, P), dtype=bool))
    off = P
    for r in branch_len:
        vis[off:off + r, :P] = True
        vis[off:off + r, off:off + r] = np.tril(np.ones((r, r), dtype=bool))
        off += r
    return vis


def masked_attention_fwd_bwd(q, k, v, do, vis, scale):
    """Dense attention under an arbitrary visibility matrix, one head.

    Every row must see at least one key.  Returns o, lse, dq, dk, dv.
    """
    s = np.where(vis, scale * (q @ k.T), -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    p = e / l
    o = p @ v
    lse = (m + np.log(l))[:, 0]
    dq, dk, dv = causal_attention_bwd(q, k, v, o, p, do, scale)
    return o, lse, dq, dk, dv


def partial_state(q, k, v, vis, scale):
    """Partial online-softmax state S = (m, l, O_acc) of queries q against one
    KV shard (Sec. 3.3, "Common tile semantics"): m the row maximum over the
    shard's visible keys, l the sum of exp(s - m), O_acc the un-normalised
    output.  A row that sees nothing in the shard gets (-inf, 0, 0).
    """
    s = np.where(vis, scale * (q @ k.T), -np.inf)
    m = s.max(axis=1) if s.shape[1] else np.full(q.shape[0], -np.inf)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    e = np.where(vis, np.exp(s - m_safe[:, None]), 0.0)
    return m, e.sum(axis=1), e @ v


def merge_states(a, b):
    """The associative merge (+) of two partial states along a query row."""
    (ma, la, oa), (mb, lb, ob) = a, b
    m = np.maximum(ma, mb)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    wa = np.where(np.isfinite(ma), np.exp(ma - m_safe), 0.0)
    wb = np.where(np.isfinite(mb), np.exp(mb - m_safe), 0.0)
    return m, wa * la + wb * lb, wa[:, None] * oa + wb[:, None] * ob


def finalize_state(state):
    """Normalised output and LSE = m + ln l of a fully merged state."""
    m, l, o = state
    return o / l[:, None], m + np.log(l)


# --------------------------------------------------------------------------- #
# Work accounting (Sec. 1: flattening recomputes (G-1)/G of the prompt work).
# --------------------------------------------------------------------------- #
def tri(n):
    return n * (n + 1) // 2


def valid_pairs(tb):
    """Visible (query, key) pairs per query head: prefill, replay, flattened."""
    prefill = replay = flat = 0
    for g in range(tb.n_groups):
        P = tb.prompt_len[g]
        prefill += tri(P)
        for r in tb.branch_len[g]:
            replay += r * P + tri(r)
            flat += tri(P + r)
        if not tb.branch_len[g]:
            flat += tri(P)
    return prefill, replay, flat
