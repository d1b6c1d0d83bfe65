"""Pins for the CPU oracle: closed forms, invariants, library routines, brute force.

Nothing here touches the CUDA path.  Each block is chosen so that a plausible slip in the oracle
(a dropped scale, a sign, a transposed operand, an off-by-one in a mask, a wrong GQA head map)
breaks at least one assertion; the ``test_pins_detect_*`` cases check that claim by feeding the
oracle deliberately wrong arguments and requiring the pin to notice.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2602_15318_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(a):
    """float array (values exactly representable or to be rounded) -> bf16 bit patterns."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).double().numpy()


def rand_bits(rng, shape):
    return bf16_bits(rng.standard_normal(shape))


def core(q, k, v, vis, scale, **kw):
    """q [T,Hq,D], k/v [Hkv,n,D], vis [T,n] -> out [T,Hq,D], lse [Hq,T] (batch of one)."""
    out, lse = oracle.attention(q[None], k[None], v[None], vis[None], [vis.shape[1]], scale, **kw)
    return out[0], lse[0]


# ---------------------------------------------------------------- closed forms ---------------

def test_hand_worked_example_eq2():
    g = json.load(open(os.path.join(GOLD, "hand_softmax_d4.json")))
    q = bf16_bits(g["q"]).reshape(1, 1, 4)
    k = bf16_bits(g["k"]).reshape(1, 3, 4)
    v = bf16_bits(g["v"]).reshape(1, 3, 4)
    out, lse = core(q, k, v, np.ones((1, 3), np.uint8), math.log(2.0))
    np.testing.assert_allclose(out[0, 0], g["out"], rtol=0, atol=1e-14)
    assert abs(lse[0, 0] - g["lse"]) < 1e-14


@pytest.mark.parametrize("D,n", [(4, 5), (128, 37)])
def test_equal_keys_give_mean_of_values(D, n):
    rng = np.random.default_rng(1)
    q = rand_bits(rng, (3, 2, D))
    krow = rand_bits(rng, (1, 1, D))
    k = np.repeat(krow, n, axis=1)
    v = rand_bits(rng, (1, n, D))
    vis = np.ones((3, n), np.uint8)
    vis[1, ::2] = 0                       # a masked row: mean over the visible subset only
    scale = 0.37
    out, lse = core(q, k, v, vis, scale)
    qf, kf, vf = bits_to_f64(q), bits_to_f64(krow)[0, 0], bits_to_f64(v)[0]
    for t in range(3):
        sel = vis[t].astype(bool)
        for h in range(2):
            s = scale * float(qf[t, h] @ kf)
            np.testing.assert_allclose(out[t, h], vf[sel].mean(axis=0), atol=1e-13)
            assert abs(lse[h, t] - (s + math.log(sel.sum()))) < 1e-12


def test_two_keys_logistic_weights():
    rng = np.random.default_rng(2)
    D = 128
    q = rand_bits(rng, (1, 1, D)); k = rand_bits(rng, (1, 2, D)); v = rand_bits(rng, (1, 2, D))
    scale = 1 / math.sqrt(D)
    out, lse = core(q, k, v, np.ones((1, 2), np.uint8), scale)
    qf, kf, vf = bits_to_f64(q)[0, 0], bits_to_f64(k)[0], bits_to_f64(v)[0]
    s = scale * (kf @ qf)
    w0 = 1.0 / (1.0 + math.exp(s[1] - s[0]))
    np.testing.assert_allclose(out[0, 0], w0 * vf[0] + (1 - w0) * vf[1], atol=1e-14)
    assert abs(lse[0, 0] - (s[0] + math.log1p(math.exp(s[1] - s[0])))) < 1e-13


def test_empty_visibility_row():
    rng = np.random.default_rng(3)
    q = rand_bits(rng, (2, 1, 8)); k = rand_bits(rng, (1, 4, 8)); v = rand_bits(rng, (1, 4, 8))
    vis = np.ones((2, 4), np.uint8); vis[1] = 0
    out, lse = core(q, k, v, vis, 1.0)
    assert np.all(out[1] == 0) and lse[0, 1] == -np.inf and np.isfinite(lse[0, 0])


# ---------------------------------------------------------------- invariants -----------------

def _case(seed, T=4, Hq=4, Hkv=2, D=16, n=24):
    rng = np.random.default_rng(seed)
    return (rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D)),
            (rng.random((T, n)) < 0.7).astype(np.uint8))


def test_score_shift_moves_lse_only():
    q, k, v, vis = _case(4)
    vis[:, 0] = 1
    T, Hq, D = q.shape
    c = 3.0
    q2 = np.concatenate([q, np.broadcast_to(bf16_bits([1.0]), (T, Hq, 1))], axis=2)
    k2 = np.concatenate([k, np.broadcast_to(bf16_bits([c]), k.shape[:2] + (1,))], axis=2)
    k0 = np.concatenate([k, np.broadcast_to(bf16_bits([0.0]), k.shape[:2] + (1,))], axis=2)
    v2 = np.concatenate([v, v[:, :, :1]], axis=2)
    scale = 0.25
    o_a, l_a = core(q2, k0, v2, vis, scale)
    o_b, l_b = core(q2, k2, v2, vis, scale)
    np.testing.assert_allclose(o_a, o_b, atol=1e-13)
    np.testing.assert_allclose(l_b - l_a, scale * c, atol=1e-12)


def test_key_permutation_invariance():
    q, k, v, vis = _case(5)
    vis[:, 0] = 1
    perm = np.random.default_rng(6).permutation(k.shape[1])
    o_a, l_a = core(q, k, v, vis, 0.3)
    o_b, l_b = core(q, k[:, perm], v[:, perm], vis[:, perm], 0.3)
    np.testing.assert_allclose(o_a, o_b, atol=1e-13)
    np.testing.assert_allclose(l_a, l_b, atol=1e-13)


def test_split_and_merge_by_logsumexp():
    """Two calls over disjoint key sets, merged by log-sum-exp, equal one call (the identity the
    split-combine step of the CUDA path relies on)."""
    q, k, v, vis = _case(7, n=30)
    vis[:, 0] = 1; vis[:, 29] = 1
    va, vb = vis.copy(), vis.copy()
    va[:, 13:] = 0; vb[:, :13] = 0
    o, l = core(q, k, v, vis, 0.3)
    oa, la = core(q, k, v, va, 0.3)
    ob, lb = core(q, k, v, vb, 0.3)
    lm = np.logaddexp(la, lb)
    wa, wb = np.exp(la - lm).T[..., None], np.exp(lb - lm).T[..., None]
    np.testing.assert_allclose(lm, l, atol=1e-12)
    np.testing.assert_allclose(wa * oa + wb * ob, o, atol=1e-12)


def test_softmax_weights_sum_to_one():
    """V = all ones (any column) -> out is exactly the sum of the weights."""
    q, k, v, vis = _case(8)
    vis[:, 3] = 1
    ones = np.broadcast_to(bf16_bits([1.0]), v.shape).copy()
    out, _ = core(q, k, ones, vis, 0.5)
    np.testing.assert_allclose(out, 1.0, atol=1e-13)


# ---------------------------------------------------------------- library routines -----------

def sdpa(q, k, v, mask, scale, G):
    """torch's float64 scaled_dot_product_attention with the KV heads repeated G times (the
    repeat_kv convention: query head h reads KV head h // G)."""
    qt = torch.from_numpy(bits_to_f64(q)).permute(1, 0, 2)[None]            # [1,Hq,T,D]
    kt = torch.from_numpy(bits_to_f64(k))[None].repeat_interleave(G, dim=1)
    vt = torch.from_numpy(bits_to_f64(v))[None].repeat_interleave(G, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


def lse_lib(q, k, mask, scale, G):
    from scipy.special import logsumexp
    qf, kf = bits_to_f64(q), np.repeat(bits_to_f64(k), G, axis=0)
    s = scale * np.einsum("thd,hjd->htj", qf, kf)
    s = np.where(mask[None], s, -np.inf)
    return logsumexp(s, axis=2)


def test_unmasked_equals_sdpa():
    rng = np.random.default_rng(10)
    T, Hq, Hkv, D, n = 5, 28, 4, 128, 300
    q, k, v = rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D))
    scale = 1 / math.sqrt(D)
    out, lse = core(q, k, v, np.ones((T, n), np.uint8), scale)
    np.testing.assert_allclose(out, sdpa(q, k, v, None, scale, 7), atol=1e-12)
    np.testing.assert_allclose(lse, lse_lib(q, k, np.ones((T, n), bool), scale, 7), atol=1e-12)


def test_chain_equals_causal_attention():
    """Chain parents [-1,0,1,..] = causal attention over kv_len+T keys, last T query rows."""
    rng = np.random.default_rng(11)
    T, Hq, Hkv, D, kv_len = 8, 28, 4, 128, 200
    n = kv_len + T
    q, k, v = rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D))
    scale = 1 / math.sqrt(D)
    parents = np.array([W.chain_parents(T)], np.int32)
    out, lse = oracle.verify_attn(q[None], k[None], v[None], [kv_len], parents, scale)
    causal = torch.ones(T, n, dtype=torch.bool).tril(diagonal=kv_len)     # bottom-right aligned
    np.testing.assert_allclose(out[0], sdpa(q, k, v, causal, scale, 7), atol=1e-12)
    np.testing.assert_allclose(lse[0], lse_lib(q, k, causal.numpy(), scale, 7), atol=1e-12)
    # square causal via the library flag: the last T rows of full causal self-attention
    qfull = np.concatenate([rand_bits(rng, (kv_len, Hq, D)), q], axis=0)
    qt = torch.from_numpy(bits_to_f64(qfull)).permute(1, 0, 2)[None]
    kt = torch.from_numpy(bits_to_f64(k))[None].repeat_interleave(7, dim=1)
    vt = torch.from_numpy(bits_to_f64(v))[None].repeat_interleave(7, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=scale)
    np.testing.assert_allclose(out[0], o[0, :, kv_len:].permute(1, 0, 2).numpy(), atol=1e-12)


def test_last_chain_node_and_forest_visibility():
    """Full-visibility readings: the last node of a chain sees every key; an all-roots forest sees
    the prefix plus itself only."""
    rng = np.random.default_rng(12)
    T, Hq, Hkv, D, kv_len = 6, 14, 2, 32, 50
    n = kv_len + T
    q, k, v = rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D))
    scale = 0.2
    out, lse = oracle.verify_attn(q[None], k[None], v[None], [kv_len],
                                  np.array([W.chain_parents(T)], np.int32), scale)
    full = sdpa(q, k, v, None, scale, 7)
    np.testing.assert_allclose(out[0, T - 1], full[T - 1], atol=1e-12)
    out_f, lse_f = oracle.verify_attn(q[None], k[None], v[None], [kv_len],
                                      np.full((1, T), -1, np.int32), scale)
    m = torch.zeros(T, n, dtype=torch.bool); m[:, :kv_len] = True
    m[torch.arange(T), kv_len + torch.arange(T)] = True
    np.testing.assert_allclose(out_f[0], sdpa(q, k, v, m, scale, 7), atol=1e-12)
    np.testing.assert_allclose(lse_f[0], lse_lib(q, k, m.numpy(), scale, 7), atol=1e-12)


def test_random_tree_equals_masked_sdpa():
    rng = np.random.default_rng(13)
    T, Hq, Hkv, D, kv_len = 12, 28, 4, 128, 77
    n = kv_len + T
    q, k, v = rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D))
    parents = W.random_tree_parents(99, 4, T, max_depth=4, max_children=3)
    mask = torch.zeros(T, n, dtype=torch.bool); mask[:, :kv_len] = True
    for t in range(T):                     # walk to the root
        a = t
        while a >= 0:
            mask[t, kv_len + a] = True
            a = parents[a]
    scale = 1 / math.sqrt(D)
    out, lse = oracle.verify_attn(q[None], k[None], v[None], [kv_len],
                                  np.array([parents], np.int32), scale)
    np.testing.assert_allclose(out[0], sdpa(q, k, v, mask, scale, 7), atol=1e-12)
    np.testing.assert_allclose(lse[0], lse_lib(q, k, mask.numpy(), scale, 7), atol=1e-12)


def test_anchored_equals_dense_on_gathered_subset():
    """Eq. 2: attention restricted to the text-anchored rows = dense attention on those rows
    copied into a compact buffer (causal among the T draft rows)."""
    rng = np.random.default_rng(14)
    T, Hq, Hkv, D = 4, 28, 4, 128
    seq_len, spans, window = 300, [[10, 250]], 0
    cap = seq_len + T
    q, k, v = rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, cap, D)), rand_bits(rng, (Hkv, cap, D))
    idx = oracle.anchor_idx(seq_len, spans, window, T)
    assert len(idx) == 10 + 50 + T
    scale = 1 / math.sqrt(D)
    out, lse = oracle.anchor_attn(q[None], k[None], v[None], idx[None], window, scale)
    kg, vg = k[:, idx], v[:, idx]
    n = len(idx)
    causal = torch.ones(T, n, dtype=torch.bool).tril(diagonal=n - T)
    np.testing.assert_allclose(out[0], sdpa(q, kg, vg, causal, scale, 7), atol=1e-12)
    np.testing.assert_allclose(lse[0], lse_lib(q, kg, causal.numpy(), scale, 7), atol=1e-12)


def test_anchored_window_lower_bound():
    rng = np.random.default_rng(15)
    T, Hq, Hkv, D = 3, 7, 1, 16
    idx = np.array([2, 5, 9, 30, 31, 40, 41, 42], np.int32)   # last 3 = draft rows
    cap = 43
    q, k, v = rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, cap, D)), rand_bits(rng, (Hkv, cap, D))
    window = 12
    vis = oracle.anchor_visibility(idx, window, T)
    want = np.array([[(p <= qp) and (qp - window < p) for p in idx] for qp in idx[-T:]], np.uint8)
    assert np.array_equal(vis, want)
    assert vis[0].tolist() == [0, 0, 0, 1, 1, 1, 0, 0]      # qpos 40: window covers 29..40
    out, lse = oracle.anchor_attn(q[None], k[None], v[None], idx[None], window, 0.3)
    np.testing.assert_allclose(out[0], sdpa(q, k[:, idx], v[:, idx], torch.from_numpy(want.astype(bool)), 0.3, 7), atol=1e-12)


def test_sampled_rows_match_full():
    case = W.make_verify_case(5, [100, 64], 5, "random")
    qb, kb, vb = W.bf16_bits(case.q), W.bf16_bits(case.k), W.bf16_bits(case.v)
    par = case.parents.numpy()
    out, lse = oracle.verify_attn(qb, kb, vb, case.kv_len, par, W.SCALE)
    rows = [(0, 0, 0), (1, 4, 27), (0, 3, 13), (1, 2, 6)]
    o2, l2 = oracle.verify_attn(qb, kb, vb, case.kv_len, par, W.SCALE, rows=rows)
    for i, (b, t, h) in enumerate(rows):
        assert np.array_equal(o2[i], out[b, t, h]) and l2[i] == lse[b, h, t]


# ---------------------------------------------------------------- masks and indices ----------

def walk_mask(parents, i):
    m, a = 0, i
    while a >= 0:
        m |= 1 << a
        a = parents[a]
    return m


def test_ancestor_masks_all_small_trees():
    for T in range(1, 7):
        for par in itertools.product(*[range(-1, i) for i in range(T)]):
            got = oracle.ancestor_masks(np.array(par, np.int32))
            assert [int(x) for x in got] == [walk_mask(par, i) for i in range(T)]


def test_ancestor_masks_closed_forms():
    T = 64
    chain = oracle.ancestor_masks(np.array(W.chain_parents(T), np.int32))
    assert [int(x) for x in chain] == [(1 << (t + 1)) - 1 for t in range(T)]
    forest = oracle.ancestor_masks(np.full(T, -1, np.int32))
    assert [int(x) for x in forest] == [1 << t for t in range(T)]
    par = W.random_tree_parents(W.config_seed(2), 4, T)
    anc = oracle.ancestor_masks(np.array(par, np.int32))
    depth = [0] * T
    for i in range(T):
        depth[i] = 1 if par[i] < 0 else depth[par[i]] + 1
    assert [bin(int(x)).count("1") for x in anc] == depth
    assert max(depth) <= 8
    assert max(par.count(j) for j in range(T)) <= 4


def test_ancestor_masks_reject_bad_trees():
    for bad in ([0], [-1, 1], [-1, 2, 0], [-2]):
        with pytest.raises(oracle.OracleError):
            oracle.ancestor_masks(np.array(bad, np.int32))


def test_verify_visibility_layout():
    anc = oracle.ancestor_masks(np.array([-1, 0, 0, 2], np.int32))
    vis = oracle.verify_visibility(3, anc)
    assert vis.shape == (4, 7)
    assert vis.tolist() == [[1, 1, 1, 1, 0, 0, 0], [1, 1, 1, 1, 1, 0, 0],
                            [1, 1, 1, 1, 0, 1, 0], [1, 1, 1, 1, 0, 1, 1]]


def _brute_force_anchor_list(seq_len, vis_spans, window, T):
    """Eq. 2's index set under the window reading, filtered position by position: every position of
    [0, seq_len) that lies in no visual span and within the last `window` positions (window <= 0:
    no limit), then the T draft rows."""
    keep = []
    for p in range(seq_len):
        visual = any(a <= p < e for a, e in vis_spans)
        recent = window <= 0 or p >= seq_len - window
        if recent and not visual:
            keep.append(p)
    return keep + [seq_len + t for t in range(T)]


def test_anchor_idx_brute_force_and_c4_closed_form():
    rng = np.random.default_rng(20)
    for _ in range(30):
        L = int(rng.integers(1, 200))
        cuts = sorted(rng.integers(0, L + 1, size=4).tolist())
        spans = [[cuts[0], cuts[1]], [cuts[2], cuts[3]]]
        Wn = int(rng.integers(0, 80)); T = int(rng.integers(0, 9))
        want = _brute_force_anchor_list(L, spans, Wn, T)
        assert oracle.anchor_idx(L, spans, Wn, T).tolist() == want
    got = oracle.anchor_idx(26112, [[64, 25664]], 1024, 8)
    assert got.tolist() == list(range(25664, 26112)) + list(range(26112, 26120))
    assert len(got) == 456
    assert oracle.anchor_idx(100, [], 0, 2).tolist() == list(range(102))


# ---------------------------------------------------------------- the pins bite --------------

def _pin_case():
    rng = np.random.default_rng(30)
    T, Hq, Hkv, D, kv_len = 6, 28, 4, 128, 90
    n = kv_len + T
    q, k, v = rand_bits(rng, (T, Hq, D)), rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D))
    causal = torch.ones(T, n, dtype=torch.bool).tril(diagonal=kv_len)
    scale = 1 / math.sqrt(D)
    return q, k, v, kv_len, causal, scale, sdpa(q, k, v, causal, scale, 7), lse_lib(q, k, causal.numpy(), scale, 7)


def _differs(a, b, tol=1e-6):
    return float(np.max(np.abs(a - b))) > tol


def test_pins_detect_planted_mistakes():
    q, k, v, kv_len, causal, scale, ref_o, ref_l = _pin_case()
    T = q.shape[0]
    chain = np.array([W.chain_parents(T)], np.int32)
    run = lambda q_, k_, v_, kl, sc, par=chain: oracle.verify_attn(q_[None], k_[None], v_[None], [kl], par, sc)
    o, l = run(q, k, v, kv_len, scale)
    assert not _differs(o[0], ref_o, 1e-12) and not _differs(l[0], ref_l, 1e-12)
    o, l = run(q, v, k, kv_len, scale)                       # K and V exchanged
    assert _differs(o[0], ref_o) and _differs(l[0], ref_l)
    o, l = run(q, k, v, kv_len, 1.0)                         # scale dropped
    assert _differs(o[0], ref_o) and _differs(l[0], ref_l)
    o, l = run(q, k, v, kv_len, -scale)                      # sign of the scores
    assert _differs(o[0], ref_o) and _differs(l[0], ref_l)
    o, l = run(q, k, v, kv_len - 1, scale)                   # off-by-one prefix
    assert _differs(o[0], ref_o) and _differs(l[0], ref_l)
    o, l = run(q[:, ::-1].copy(), k, v, kv_len, scale)       # wrong query-head -> KV-head map
    assert _differs(o[0], ref_o) and _differs(l[0], ref_l)
    o, l = run(q, k, v, kv_len, scale, np.full((1, T), -1, np.int32))   # tree mask ignored
    assert _differs(o[0], ref_o) and _differs(l[0], ref_l)
    o, l = run(q[::-1].copy(), k, v, kv_len, scale)          # token order reversed
    assert _differs(o[0], ref_o) and _differs(l[0], ref_l)


# ---- tree-structured draft tokens in the anchored mode ------------------------------------------

def _walk_is_ancestor_or_self(parents, i, a):
    while i >= 0:
        if i == a:
            return True
        i = parents[i]
    return False


def test_anchor_tree_visibility_chain_reduces_to_chain_mode():
    idx = np.array([3, 4, 9, 40, 41, 77, 100, 101, 102, 103, 104], dtype=np.int32)
    T = 5
    chain = np.arange(-1, T - 1, dtype=np.int32)
    for window in (0, 64, 1000):          # windows wider than the draft block: the two rules coincide
        assert np.array_equal(oracle.anchor_tree_visibility(idx, window, chain, T),
                              oracle.anchor_visibility(idx, window, T))


def test_anchor_tree_visibility_brute_force():
    rng = np.random.default_rng(5)
    for trial in range(30):
        Tt = int(rng.integers(1, 13))
        T_new = int(rng.integers(1, Tt + 1))
        n_text = int(rng.integers(0, 20))
        rows = np.sort(rng.choice(500, size=n_text, replace=False)).astype(np.int32)
        idx = np.concatenate([rows, 600 + np.arange(Tt, dtype=np.int32)])
        parents = np.array([int(rng.integers(-1, i)) for i in range(Tt)], dtype=np.int32)
        window = int(rng.choice([0, 50, 300]))
        vis = oracle.anchor_tree_visibility(idx, window, parents, T_new)
        for t in range(T_new):
            node = Tt - T_new + t
            qpos = 600 + node
            for j in range(n_text):
                expect = rows[j] <= qpos and (window <= 0 or rows[j] > qpos - window)
                assert vis[t, j] == int(expect)
            for a in range(Tt):
                assert vis[t, n_text + a] == int(_walk_is_ancestor_or_self(parents.tolist(), node, a))


def test_anchor_tree_on_contiguous_rows_equals_verification():
    """With every row an anchor and no window, the anchored mode with a tree is the verification
    mode (whole prefix + ancestors): pins the tree variant to the oracle of mode (a), including the
    node offset when only the last nodes are queries."""
    case = W.make_verify_case(77, [37, 20], 9, "random", "cpu")
    q, k, v = W.bf16_bits(case.q), W.bf16_bits(case.k), W.bf16_bits(case.v)
    par = case.parents.numpy()
    ref_out, ref_lse = oracle.verify_attn(q, k, v, case.kv_len, par, W.SCALE)
    for b in range(case.B):
        n = case.kv_len[b] + case.T
        idx = np.arange(n, dtype=np.int32)[None]
        for T_new in (case.T, 4, 1):
            qb = q[b:b + 1, case.T - T_new:]
            out, lse = oracle.anchor_attn_tree(qb, k[b:b + 1], v[b:b + 1], idx, 0, par[b:b + 1], W.SCALE)
            assert np.allclose(out[0], ref_out[b, case.T - T_new:], atol=1e-12)
            assert np.allclose(lse[0], ref_lse[b][:, case.T - T_new:], atol=1e-12)


def test_anchor_tree_forest_of_roots_sees_text_and_itself_only():
    idx = np.array([1, 2, 5, 50, 51, 52], dtype=np.int32)
    vis = oracle.anchor_tree_visibility(idx, 0, np.array([-1, -1, -1], dtype=np.int32), 3)
    assert np.array_equal(vis[:, :3], np.ones((3, 3), dtype=np.uint8))
    assert np.array_equal(vis[:, 3:], np.eye(3, dtype=np.uint8))


# ---- greedy acceptance of a draft tree -----------------------------------------------------------

def _accepted_paths_brute_force(tok, par, nxt):
    """Every node whose whole chain from its root matches the target, found by walking up from the
    node and checking each step on its own (independent of the oracle's forward recurrence)."""
    good = []
    for i in range(len(tok)):
        chain, n = [], i
        while n >= 0:
            chain.append(n)
            n = par[n]
        chain.reverse()
        if all(tok[c] == nxt[par[c] + 1] for c in chain):
            good.append(chain)
    return good


def test_greedy_accept_brute_force_on_random_trees():
    rng = np.random.default_rng(11)
    for trial in range(300):
        T = int(rng.integers(1, 12))
        par = [int(rng.integers(-1, i)) for i in range(T)]
        nxt = [int(rng.integers(0, 3)) for _ in range(T + 1)]
        tok = [int(rng.integers(0, 3)) for _ in range(T)]
        path, bonus = oracle.greedy_accept(tok, par, nxt)
        good = _accepted_paths_brute_force(tok, par, nxt)
        if not good:
            assert path == [] and bonus == nxt[0]
            continue
        longest = max(len(c) for c in good)
        expect = min((c for c in good if len(c) == longest), key=lambda c: c[-1])
        assert path == expect and bonus == nxt[expect[-1] + 1]


def test_greedy_accept_closed_forms():
    chain = [-1, 0, 1, 2, 3]
    nxt = [7, 8, 9, 10, 11, 12]
    assert oracle.greedy_accept([7, 8, 9, 10, 11], chain, nxt) == ([0, 1, 2, 3, 4], 12)     # everything matches
    assert oracle.greedy_accept([7, 8, 0, 10, 11], chain, nxt) == ([0, 1], 9)               # first mismatch cuts the chain
    assert oracle.greedy_accept([0, 8, 9, 10, 11], chain, nxt) == ([], 7)                   # nothing accepted: the target's own token
    # two roots, the second one right; its two children compete, the deeper branch wins
    par = [-1, -1, 1, 1, 3]
    assert oracle.greedy_accept([5, 7, 8, 8, 4], par, [7, 0, 8, 0, 4, 6]) == ([1, 3, 4], 6)
    # equal depth: the chain ending at the smaller index
    assert oracle.greedy_accept([5, 7, 8, 8, 1], par, [7, 0, 8, 0, 4, 6]) == ([1, 2], 0)


# ---------------------------------------------------------------- acceptance at temperature 1 ----
# Pinned by what speculative sampling must satisfy whatever the implementation: identical draft and
# target distributions accept everything, disjoint supports accept nothing, a one-hot target is
# the greedy rule, and the emitted tokens follow the target distribution exactly (checked
# empirically with siblings drawn without replacement from the draft distribution).

def _rows(rng, n_rows, V, conc=1.0):
    return rng.dirichlet([conc] * V, size=n_rows).astype(np.float32)


def _uniforms(rng, n):
    return rng.integers(0, 1 << 32, size=n, dtype=np.uint64)


def test_sample_accept_identical_distributions_accept_the_first_child_chain():
    rng = np.random.default_rng(41)
    for _ in range(20):
        T, V = int(rng.integers(1, 12)), 17
        par = W.random_tree_parents(int(rng.integers(1 << 30)), 3, T)
        p = _rows(rng, T + 1, V)
        # any token with draft probability > 0 is accepted, whatever the uniform says
        tok = [int(rng.choice(np.flatnonzero(p[par[i] + 1] > 1e-6))) for i in range(T)]
        path, bonus = oracle.sample_accept(tok, par, p, p, _uniforms(rng, T), _uniforms(rng, T + 1))
        want, cur = [], -1
        while True:
            kids = [i for i in range(T) if par[i] == cur]
            if not kids:
                break
            cur = kids[0]
            want.append(cur)
        assert path == want and 0 <= bonus < V


def test_sample_accept_disjoint_supports_accept_nothing_and_emit_from_the_target():
    rng = np.random.default_rng(42)
    V, T, n = 8, 3, 4000
    p = np.zeros((T + 1, V), np.float32); q = np.zeros_like(p)
    p[:, :4] = _rows(rng, T + 1, 4); q[:, 4:] = _rows(rng, T + 1, 4)
    counts = np.zeros(V)
    for _ in range(n):
        tok = [int(rng.integers(4, 8)) for _ in range(T)]
        path, bonus = oracle.sample_accept(tok, [-1, -1, 0], p, q, _uniforms(rng, T), _uniforms(rng, T + 1))
        assert path == []
        counts[bonus] += 1
    assert counts[4:].sum() == 0
    expect = p[0].astype(np.float64) * n
    assert np.all(np.abs(counts[:4] - expect[:4]) < 5 * np.sqrt(expect[:4] + 1))


def test_sample_accept_with_one_hot_target_is_the_greedy_rule():
    rng = np.random.default_rng(43)
    for _ in range(30):
        T, V = int(rng.integers(1, 14)), 6
        par = W.random_tree_parents(int(rng.integers(1 << 30)), 5, T)
        nxt = rng.integers(0, V, size=T + 1)
        p = np.zeros((T + 1, V), np.float32)
        p[np.arange(T + 1), nxt] = 1.0
        q = _rows(rng, T + 1, V) * 0.98 + 0.02 / V           # every token has draft mass
        tok = []
        for i in range(T):                                   # siblings carry distinct tokens
            used = {tok[j] for j in range(i) if par[j] == par[i]}
            tok.append(int(rng.choice([v for v in range(V) if v not in used])))
        path, bonus = oracle.sample_accept(tok, par, p, q, _uniforms(rng, T), _uniforms(rng, T + 1))
        g_path, g_bonus = oracle.greedy_accept(tok, par, nxt)
        # the walk follows accepted children, so it is the greedy chain whenever that chain is unique
        # (distinct sibling tokens: at most one child of a node can match the target's token)
        assert path == g_path and bonus == g_bonus


def _draw_children_without_replacement(rng, q_row, k):
    q = q_row.astype(np.float64).copy()
    out = []
    for _ in range(k):
        q /= q.sum()
        x = int(rng.choice(len(q), p=q))
        out.append(x)
        q[x] = 0.0
    return out


def test_sample_accept_emits_the_target_distribution():
    """Root level with up to 3 sibling candidates drawn without replacement from q, then one more
    level below the first candidate: the first and the second emitted token must be distributed as
    the target rows say, although target and draft differ a lot."""
    rng = np.random.default_rng(44)
    V, n = 4, 30000
    par = [-1, -1, -1, 0, 0]
    p = np.array([[0.55, 0.05, 0.30, 0.10], [0.10, 0.60, 0.10, 0.20], [0.25, 0.25, 0.25, 0.25],
                  [0.70, 0.10, 0.10, 0.10], [0.40, 0.30, 0.20, 0.10], [0.10, 0.20, 0.30, 0.40]], np.float32)
    q = np.array([[0.10, 0.40, 0.20, 0.30], [0.30, 0.20, 0.40, 0.10], [0.25, 0.25, 0.25, 0.25],
                  [0.25, 0.25, 0.25, 0.25], [0.25, 0.25, 0.25, 0.25], [0.25, 0.25, 0.25, 0.25]], np.float32)
    first = np.zeros(V)
    second_after_node0 = np.zeros(V)
    n_node0 = 0
    for _ in range(n):
        roots = _draw_children_without_replacement(rng, q[0], 3)
        kids = _draw_children_without_replacement(rng, q[1], 2)
        tok = roots + kids
        path, bonus = oracle.sample_accept(tok, par, p, q, _uniforms(rng, 5), _uniforms(rng, 6))
        emitted = [tok[i] for i in path] + [bonus]
        first[emitted[0]] += 1
        if path and path[0] == 0:                           # the walk went through node 0: row 1 is next
            n_node0 += 1
            second_after_node0[emitted[1]] += 1
    e1 = p[0].astype(np.float64) * n
    assert np.all(np.abs(first - e1) < 4.5 * np.sqrt(e1)), (first, e1)
    assert n_node0 > 2000
    # the token after node 0 follows the target row of node 0 whatever token node 0 carried
    e2 = p[1].astype(np.float64) * n_node0
    assert np.all(np.abs(second_after_node0 - e2) < 4.5 * np.sqrt(e2)), (second_after_node0, e2)


def test_sample_accept_pin_detects_a_planted_mistake():
    """The distribution pin bites: leaving the draft distribution untouched after a rejection (the
    with-replacement rule applied to candidates drawn without replacement) shifts the output."""
    rng = np.random.default_rng(45)
    V, n = 4, 30000
    p = np.array([[0.55, 0.05, 0.30, 0.10]] * 4, np.float32)
    q = np.array([[0.10, 0.40, 0.20, 0.30]] * 4, np.float32)

    def wrong(tok, u_node, u_bonus):                        # the oracle's steps with the planted mistake
        P, Q = oracle.fixed_point_probs(p[0]), oracle.fixed_point_probs(q[0])
        A, Bq = int(P.sum()), int(Q.sum())
        for c, x in enumerate(tok):
            if int(u_node[c]) * int(Q[x]) * A < int(P[x]) * Bq * (1 << 32):
                return x
            P = np.maximum(Bq * P - A * Q, 0) >> 30
            A = int(P.sum())                                # Q keeps x: the mistake
        t = (int(u_bonus[0]) * A) >> 32
        return int(np.searchsorted(np.cumsum(P), t, side="right"))

    counts = np.zeros(V)
    for _ in range(n):
        tok = _draw_children_without_replacement(rng, q[0], 3)
        counts[wrong(tok, _uniforms(rng, 3), _uniforms(rng, 1))] += 1
    e = p[0].astype(np.float64) * n
    assert np.any(np.abs(counts - e) > 6 * np.sqrt(e))


# ---------------------------------------------------------------- hidden-state reuse (Eq. 1) ----

def _bits(a):
    return W.bf16_bits(torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def test_hsr_fuse_hand_worked_example():
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hsr_fuse_small.json")))
    z = oracle.hsr_fuse(_bits(g["e"]), _bits(g["h"]), _bits(g["w"]), _bits(g["bias"]))
    assert np.array_equal(z, np.array(g["z"]))
    z0 = oracle.hsr_fuse(_bits(g["e"]), _bits(g["h"]), _bits(g["w"]))
    assert np.array_equal(z0, np.array(g["z_without_bias"]))


def test_hsr_fuse_selector_weights_pick_the_two_halves():
    """W = [I | 0] returns e, W = [0 | I] returns h, W = [I | I] their sum: the concatenation puts
    the embedding first and the hidden state second."""
    rng = np.random.default_rng(50)
    M, d = 5, 16
    e, h = rand_bits(rng, (M, d)), rand_bits(rng, (M, d))
    E, H = oracle.bf16_bits_to_f64(e), oracle.bf16_bits_to_f64(h)
    I, Z = np.eye(d), np.zeros((d, d))
    assert np.array_equal(oracle.hsr_fuse(e, h, _bits(np.hstack([I, Z]))), E)
    assert np.array_equal(oracle.hsr_fuse(e, h, _bits(np.hstack([Z, I]))), H)
    assert np.array_equal(oracle.hsr_fuse(e, h, _bits(np.hstack([I, I]))), E + H)
    assert not np.array_equal(E, H)


def test_hsr_fuse_brute_force_and_library_linear():
    rng = np.random.default_rng(51)
    M, d, n = 3, 8, 6
    e, h, w, b = rand_bits(rng, (M, d)), rand_bits(rng, (M, d)), rand_bits(rng, (n, 2 * d)), rand_bits(rng, (n,))
    z = oracle.hsr_fuse(e, h, w, b)
    E, H, Wt, Bv = (oracle.bf16_bits_to_f64(a) for a in (e, h, w, b))
    for m in range(M):                              # the definition, term by term
        for o in range(n):
            acc = Bv[o]
            for k in range(d):
                acc += E[m, k] * Wt[o, k]
            for k in range(d):
                acc += H[m, k] * Wt[o, d + k]
            assert abs(z[m, o] - acc) <= 1e-12 * (1 + abs(acc))
    lib = torch.nn.functional.linear(torch.cat([torch.from_numpy(E), torch.from_numpy(H)], dim=1),
                                     torch.from_numpy(Wt), torch.from_numpy(Bv)).numpy()
    assert np.max(np.abs(z - lib)) <= 1e-12
