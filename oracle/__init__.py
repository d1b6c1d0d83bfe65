"""CPU oracle for the Sparrow speculative-step attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes marshalling around ``sparrow_oracle.c`` (plain C, fp64).  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import this package; the product never does.
Arrays are numpy: bf16 tensors travel as ``uint16`` bit patterns, results come back as float64.
"""
import ctypes
import os

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(_build.build())
        i32, i64, f64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        L.oracle_ancestor_masks.argtypes = [vp, i32, vp]
        L.oracle_verify_visibility.argtypes = [i32, i32, vp, vp, i64]
        L.oracle_anchor_idx.argtypes = [i32, vp, i32, i32, i32, vp, vp]
        L.oracle_anchor_visibility.argtypes = [vp, i32, i32, i32, vp, i64]
        L.oracle_attention.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32,
                                       i64, i64, f64, vp, i64, i32, vp, vp]
        L.oracle_verify_attn.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32,
                                         i64, i64, f64, vp, i64, i32, vp, vp]
        L.oracle_anchor_attn.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                         i64, i64, f64, vp, i64, i32, vp, vp]
        for f in ("oracle_ancestor_masks", "oracle_verify_visibility", "oracle_anchor_idx",
                  "oracle_anchor_visibility", "oracle_attention", "oracle_verify_attn",
                  "oracle_anchor_attn"):
            getattr(L, f).restype = ctypes.c_int
        _lib = L
    return _lib


class OracleError(RuntimeError):
    pass


def _chk(rc, what):
    if rc != 0:
        raise OracleError(f"{what} failed with oracle status {rc}")


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def host_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def ancestor_masks(parents) -> np.ndarray:
    """parents: int32 [T] -> uint64 [T]; bit a of entry i set iff a == i or a is an ancestor of i."""
    parents = _c(parents, np.int32)
    T = parents.shape[0]
    anc = np.zeros(max(T, 1), dtype=np.uint64)
    _chk(lib().oracle_ancestor_masks(_p(parents), T, _p(anc)), "oracle_ancestor_masks")
    return anc[:T]


def verify_visibility(kv_len: int, anc) -> np.ndarray:
    anc = _c(anc, np.uint64)
    T = anc.shape[0]
    vis = np.zeros((T, kv_len + T), dtype=np.uint8)
    _chk(lib().oracle_verify_visibility(kv_len, T, _p(anc), _p(vis), vis.shape[1]),
         "oracle_verify_visibility")
    return vis


def anchor_idx(seq_len: int, vis_spans, window: int, T: int) -> np.ndarray:
    spans = _c(np.asarray(vis_spans, dtype=np.int32).reshape(-1, 2), np.int32)
    idx = np.zeros(seq_len + T + 1, dtype=np.int32)
    n = ctypes.c_int32(0)
    _chk(lib().oracle_anchor_idx(seq_len, _p(spans) if spans.size else None, spans.shape[0],
                                 window, T, _p(idx), ctypes.byref(n)), "oracle_anchor_idx")
    return idx[: n.value].copy()


def anchor_visibility(idx, window: int, T: int) -> np.ndarray:
    idx = _c(idx, np.int32)
    n = idx.shape[0]
    vis = np.zeros((T, n), dtype=np.uint8)
    _chk(lib().oracle_anchor_visibility(_p(idx), n, window, T, _p(vis), n),
         "oracle_anchor_visibility")
    return vis


def _rows_arg(rows):
    if rows is None:
        return None, 0
    rows = _c(np.asarray(rows).reshape(-1, 3), np.int32)
    return rows, rows.shape[0]


def _outs(rows, n_rows, B, T, Hq, D):
    if rows is None:
        return np.zeros((B, T, Hq, D)), np.zeros((B, Hq, T))
    return np.zeros((n_rows, D)), np.zeros((n_rows,))


def _kv_strides(k, B, Hkv, D):
    assert k.ndim == 4 and k.shape[0] == B and k.shape[1] == Hkv and k.shape[3] == D
    assert k.flags.c_contiguous
    return k.shape[1] * k.shape[2] * D, k.shape[2] * D


def attention(q, k, v, vis, n_keys_b, scale, key_rows=None, rows=None, n_threads=None):
    """Core: q uint16 [B,T,Hq,D]; k,v uint16 [B,Hkv,cap,D]; vis uint8 [B,T,n_keys]."""
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    vis = _c(vis, np.uint8)
    B, T, Hq, D = q.shape
    Hkv = k.shape[1]
    n_keys = vis.shape[2]
    nk = _c(n_keys_b, np.int32)
    sb, sh = _kv_strides(k, B, Hkv, D)
    assert v.shape == k.shape
    if key_rows is not None:
        key_rows = _c(key_rows, np.int32)
        assert key_rows.shape == (B, n_keys)
        assert key_rows.size == 0 or (key_rows.min() >= 0 and key_rows.max() < k.shape[2])
    else:
        assert n_keys <= k.shape[2]
    rows_a, n_rows = _rows_arg(rows)
    out, lse = _outs(rows_a, n_rows, B, T, Hq, D)
    _chk(lib().oracle_attention(_p(q), _p(k), _p(v), _p(key_rows), _p(vis), _p(nk), B, T, Hq, Hkv,
                                D, n_keys, sb, sh, float(scale), _p(rows_a), n_rows,
                                n_threads or host_threads(), _p(out), _p(lse)), "oracle_attention")
    return out, lse


def verify_attn(q, k_cache, v_cache, kv_len, parents, scale, rows=None, n_threads=None):
    """Verification mode. parents int32 [B,T]; kv_len int32 [B]. Returns (out f64, lse f64)."""
    q, k, v = _c(q, np.uint16), _c(k_cache, np.uint16), _c(v_cache, np.uint16)
    B, T, Hq, D = q.shape
    Hkv = k.shape[1]
    kv_len = _c(kv_len, np.int32)
    parents = _c(parents, np.int32)
    assert kv_len.shape == (B,) and parents.shape == (B, T)
    assert int(kv_len.max()) + T <= k.shape[2]
    sb, sh = _kv_strides(k, B, Hkv, D)
    rows_a, n_rows = _rows_arg(rows)
    out, lse = _outs(rows_a, n_rows, B, T, Hq, D)
    _chk(lib().oracle_verify_attn(_p(q), _p(k), _p(v), _p(kv_len), _p(parents), B, T, Hq, Hkv, D,
                                  sb, sh, float(scale), _p(rows_a), n_rows,
                                  n_threads or host_threads(), _p(out), _p(lse)),
         "oracle_verify_attn")
    return out, lse


def anchor_attn(q, k, v, idx, window, scale, rows=None, n_threads=None):
    """Text-anchored window mode. idx int32 [B,n_anchor]; T = q.shape[1]."""
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    B, T, Hq, D = q.shape
    Hkv = k.shape[1]
    idx = _c(idx, np.int32)
    assert idx.ndim == 2 and idx.shape[0] == B
    assert idx.size == 0 or (idx.min() >= 0 and idx.max() < k.shape[2])
    sb, sh = _kv_strides(k, B, Hkv, D)
    rows_a, n_rows = _rows_arg(rows)
    out, lse = _outs(rows_a, n_rows, B, T, Hq, D)
    _chk(lib().oracle_anchor_attn(_p(q), _p(k), _p(v), _p(idx), idx.shape[1], window, B, T, Hq,
                                  Hkv, D, sb, sh, float(scale), _p(rows_a), n_rows,
                                  n_threads or host_threads(), _p(out), _p(lse)),
         "oracle_anchor_attn")
    return out, lse


def anchor_tree_visibility(idx, window: int, parents, T_new: int) -> np.ndarray:
    """Visibility of text-anchored attention whose draft tokens form a tree (the paper drafts a
    dynamic tree, Section 4 "Implementation"; Eq. 2 itself is written for one chain step).

    idx int32 [n_anchor], strictly increasing; its last T_tree = len(parents) entries are the rows
    of the tree's nodes, node i at idx[n_anchor - T_tree + i].  The queries are the last T_new
    nodes.  Query node i (row qpos) sees
      * a text anchor p (any of the first n_anchor - T_tree entries) iff p <= qpos and
        (window <= 0 or qpos - window < p): the rule of the chain mode;
      * a tree node a iff a == i or a is an ancestor of i.
    Returns uint8 [T_new, n_anchor].  Written out directly from this definition (numpy loops)."""
    idx = _c(idx, np.int32)
    parents = _c(parents, np.int32)
    n, Tt = idx.shape[0], parents.shape[0]
    assert 1 <= T_new <= Tt <= n
    anc = ancestor_masks(parents)
    first = n - Tt
    vis = np.zeros((T_new, n), dtype=np.uint8)
    for t in range(T_new):
        node = Tt - T_new + t
        qpos = int(idx[first + node])
        for j in range(first):
            p = int(idx[j])
            vis[t, j] = 1 if (p <= qpos and (window <= 0 or qpos - window < p)) else 0
        for a in range(Tt):
            vis[t, first + a] = (int(anc[node]) >> a) & 1
    return vis


def anchor_attn_tree(q, k, v, idx, window, parents, scale, rows=None, n_threads=None):
    """Text-anchored attention with tree-structured draft tokens.  q uint16 [B,T_new,Hq,D];
    idx int32 [B,n_anchor]; parents int32 [B,T_tree].  The definition of the attention itself is
    the core's (Eq. 2 on the gathered rows); only the visibility differs from anchor_attn()."""
    q = _c(q, np.uint16)
    idx = _c(idx, np.int32)
    parents = _c(parents, np.int32)
    B, T_new = q.shape[0], q.shape[1]
    assert idx.shape[0] == B and parents.shape[0] == B
    vis = np.stack([anchor_tree_visibility(idx[b], window, parents[b], T_new) for b in range(B)])
    return attention(q, k, v, vis, np.full(B, idx.shape[1], dtype=np.int32), scale, key_rows=idx,
                     rows=rows, n_threads=n_threads)


def greedy_accept(draft_tokens, parents, target_next):
    """Greedy (temperature 0) verification of a draft tree (Appendix A, "Speculative Decoding": the
    target checks the candidates of the tree in one forward pass and keeps what it would have
    produced itself, which is what makes the method lossless).

    draft_tokens int [T]; parents int [T] (-1 = root, parents[i] < i); target_next int [T + 1]:
    target_next[0] is the target's own next token after the committed prefix, target_next[1 + i]
    its next token after node i.  A node is accepted iff its token is what the target produces
    after its parent (after the prefix, for a root) and its parent is accepted.  Returns
    (path, bonus): the nodes of the deepest accepted chain from its root down (ties: the chain
    whose last node has the smallest index) and the target's token after the chain's last node
    (target_next[0] when nothing is accepted).  Plain loops, straight from this definition."""
    tok = [int(x) for x in draft_tokens]
    par = [int(x) for x in parents]
    nxt = [int(x) for x in target_next]
    T = len(tok)
    assert len(par) == T and len(nxt) == T + 1
    accepted, depth = [False] * T, [0] * T
    for i in range(T):
        p = par[i]
        assert -1 <= p < i
        ok_parent = True if p < 0 else accepted[p]
        accepted[i] = ok_parent and tok[i] == nxt[p + 1]
        depth[i] = (0 if p < 0 else depth[p]) + 1 if accepted[i] else 0
    best = -1
    for i in range(T):
        if accepted[i] and (best < 0 or depth[i] > depth[best]):
            best = i
    path = []
    i = best
    while i >= 0:
        path.append(i)
        i = par[i]
    path.reverse()
    return path, nxt[best + 1]


# ---------------------------------------------------------------------------------------------
# Acceptance at temperature 1 (speculative sampling over a draft tree).
#
# Appendix A ("Speculative Decoding") states that verification keeps the target model's output
# distribution exactly and Section 4 reports every result at temperature 0 and 1; the paper relies
# on the standard procedure without restating it.  The reading taken here is the usual multi-round
# rejection rule for a tree whose sibling candidates were drawn without replacement from the
# draft distribution: at the current node, with target distribution p and draft distribution q,
# the children are tried in index order; a child with token x is accepted with probability
# min(1, p(x) / q(x)); after a rejection p becomes the normalised positive part of (p - q) and q
# loses x and is renormalised; when no child is accepted the next token is drawn from what p has
# become.  Accepting a child moves to it, with that node's own p and q.
#
# The result is a set of integers (accepted path, bonus token), so the arithmetic that decides
# them is fixed to something every implementation reproduces bit for bit: probabilities are
# rounded once to 30-bit fixed point and everything after that is integer arithmetic, whose sums
# do not depend on the order of summation.
# ---------------------------------------------------------------------------------------------

PROB_BITS = 30


def fixed_point_probs(p) -> np.ndarray:
    """float32 probabilities -> int64 fixed point: floor(p * 2^30 + 1/2), evaluated in float64
    (exact for float32 inputs in [0, 1])."""
    p = np.asarray(p, dtype=np.float32).astype(np.float64)
    assert np.all(p >= 0.0) and np.all(p <= 1.0)
    return np.floor(p * float(1 << PROB_BITS) + 0.5).astype(np.int64)


def sample_accept(draft_tokens, parents, p_target, p_draft, u_node, u_bonus):
    """Temperature-1 verification of one draft tree.

    draft_tokens int [T]; parents int [T] (-1 = root, parents[i] < i);
    p_target, p_draft float32 [T + 1][V]: row 0 belongs to the committed prefix, row 1 + i to node
    i -- the target's next-token distribution there, and the draft distribution that node's
    children were drawn from (without replacement, in index order);
    u_node uint32 [T]: the uniform that decides node i's acceptance test;
    u_bonus uint32 [T + 1]: row r's uniform for the token drawn when the walk stops at row r.
    Returns (path, bonus): accepted nodes from the root down, and the token emitted after them.

    With P, Q the fixed-point rows (int), A = sum P, B = sum Q and r = u_node[c] in [0, 2^32):
      accept child c (token x)  iff  Q[x] > 0 and r * Q[x] * A < P[x] * B * 2^32
                                     (i.e. r / 2^32 < (P[x] / A) / (Q[x] / B));
      after a rejection         P <- max(B * P - A * Q, 0) >> 30  (element-wise; left as it is when B == 0),
                                A <- sum P,  B <- B - Q[x],  Q[x] <- 0;
      bonus                     the smallest v with P[0] + ... + P[v] > (u_bonus[row] * A) >> 32,
                                P being the row's original target row again if A == 0.
    """
    tok = [int(x) for x in draft_tokens]
    par = [int(x) for x in parents]
    T = len(tok)
    p_target = np.asarray(p_target, dtype=np.float32)
    p_draft = np.asarray(p_draft, dtype=np.float32)
    assert p_target.shape == p_draft.shape and p_target.shape[0] == T + 1
    assert len(par) == T and len(u_node) == T and len(u_bonus) == T + 1
    children = {i: [] for i in range(-1, T)}
    for i, p in enumerate(par):
        assert -1 <= p < i
        children[p].append(i)
    cur, path = -1, []
    while True:
        row = cur + 1
        P = fixed_point_probs(p_target[row])
        Q = fixed_point_probs(p_draft[row])
        A, B = int(P.sum()), int(Q.sum())
        taken = None
        for c in children[cur]:
            x, r = tok[c], int(u_node[c])
            assert 0 <= x < P.shape[0] and 0 <= r < (1 << 32)
            if int(Q[x]) > 0 and r * int(Q[x]) * A < int(P[x]) * B * (1 << 32):
                taken = c
                break
            if B > 0:
                P = np.maximum(B * P - A * Q, 0) >> PROB_BITS
                A = int(P.sum())
            B -= int(Q[x])
            Q[x] = 0
        if taken is None:
            if A == 0:
                P = fixed_point_probs(p_target[row])
                A = int(P.sum())
            assert A > 0, "a target row without any probability mass"
            t = (int(u_bonus[row]) * A) >> 32
            acc, bonus = 0, None
            for v in range(P.shape[0]):
                acc += int(P[v])
                if acc > t:
                    bonus = v
                    break
            return path, bonus
        path.append(taken)
        cur = taken


# ---------------------------------------------------------------------------------------------
# Hidden-state reuse: the draft model's input (Section 3.1, Eq. 1)
#     z_t = FC(e_t (+) h_t),
# the projection FC applied to the concatenation of the token embedding e_t and the target model's
# hidden state h_t (of its second-to-last layer, at the previous position) -- 2 d features down to
# d.  FC is taken as an ordinary linear layer, z = W x + b with W of shape [d_out][2 d] (the layout
# of torch.nn.Linear); the paper does not say whether it has a bias, so the bias is optional.
# ---------------------------------------------------------------------------------------------

def bf16_bits_to_f64(bits) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64, exactly (a bf16 is the top half of a float32)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def hsr_fuse(e, h, w, bias=None) -> np.ndarray:
    """e, h: uint16 bf16 bits [M][d]; w: bits [d_out][2 d]; bias: bits [d_out] or None.
    Returns z float64 [M][d_out] = concat(e, h) @ w.T (+ bias), all in float64."""
    E, H, Wt = bf16_bits_to_f64(e), bf16_bits_to_f64(h), bf16_bits_to_f64(w)
    assert E.ndim == 2 and E.shape == H.shape and Wt.ndim == 2 and Wt.shape[1] == 2 * E.shape[1]
    x = np.concatenate([E, H], axis=1)                 # e (+) h
    z = x @ Wt.T
    if bias is not None:
        b = bf16_bits_to_f64(bias)
        assert b.shape == (Wt.shape[0],)
        z = z + b[None, :]
    return z
