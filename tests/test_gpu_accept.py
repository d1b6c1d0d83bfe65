"""Greedy acceptance of a draft tree and the move of the accepted K/V rows, through the C ABI,
bit-exact against the oracle (integer work: no tolerance)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_15318_b200 import binding as B
from paper_2602_15318_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _random_problem(seed, batch, T, vocab):
    g = W.host_stream(seed, 55)
    par = [W.random_tree_parents(seed + 17 * b, 56, T) for b in range(batch)]
    nxt = [[next(g) % vocab for _ in range(T + 1)] for _ in range(batch)]
    tok = []
    for b in range(batch):
        row = []
        for i in range(T):
            right = nxt[b][par[b][i] + 1]
            row.append(right if next(g) % 3 else (right + 1) % vocab)      # two in three guesses are right
        tok.append(row)
    return tok, par, nxt


@pytest.mark.parametrize("batch,T,vocab", [(1, 1, 5), (1, 30, 4), (3, 48, 3), (8, 64, 2), (64, 9, 6)])
def test_accept_greedy_matches_the_oracle(batch, T, vocab):
    tok, par, nxt = _random_problem(9000 + batch + T, batch, T, vocab)
    case = W.make_verify_case(9100, [40] * batch, T, "chain", DEV)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    d = lambda x: torch.tensor(x, dtype=torch.int32, device=DEV)
    path = torch.full((batch, T), 99, dtype=torch.int32, device=DEV)
    n_acc = torch.full((batch,), 99, dtype=torch.int32, device=DEV)
    bonus = torch.full((batch,), 99, dtype=torch.int32, device=DEV)
    B.sparrow_accept_greedy(ctx, d(tok), d(par), d(nxt), T, path, n_acc, bonus)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    for b in range(batch):
        ref_path, ref_bonus = oracle.greedy_accept(tok[b], par[b], nxt[b])
        assert int(n_acc[b]) == len(ref_path)
        assert path[b].tolist() == ref_path + [-1] * (T - len(ref_path))
        assert int(bonus[b]) == ref_bonus


def test_accept_then_keep_moves_exactly_the_accepted_rows():
    batch, T = 3, 20
    tok, par, nxt = _random_problem(9300, batch, T, 3)
    case = W.make_verify_case(9301, [100, 7, 333], T, "chain", DEV, capacity=400)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    d = lambda x: torch.tensor(x, dtype=torch.int32, device=DEV)
    path = torch.empty((batch, T), dtype=torch.int32, device=DEV)
    n_acc = torch.empty((batch,), dtype=torch.int32, device=DEV)
    bonus = torch.empty((batch,), dtype=torch.int32, device=DEV)
    k0, v0 = case.k.clone(), case.v.clone()
    B.sparrow_accept_greedy(ctx, d(tok), d(par), d(nxt), T, path, n_acc, bonus)
    B.sparrow_kv_keep_accepted(ctx, case.k, case.v, case.kv_len, path, n_acc, T)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    orig_k, orig_v = k0.clone(), v0.clone()
    for b, n in enumerate(case.kv_len):
        ref_path, _ = oracle.greedy_accept(tok[b], par[b], nxt[b])
        for i, node in enumerate(ref_path):                  # all sources are the rows as they were before the call
            k0[b, :, n + i] = orig_k[b, :, n + node]
            v0[b, :, n + i] = orig_v[b, :, n + node]
    # rows of accepted nodes moved to the front of the draft block; everything else untouched
    for b, n in enumerate(case.kv_len):
        ref_path, _ = oracle.greedy_accept(tok[b], par[b], nxt[b])
        m = len(ref_path)
        assert torch.equal(case.k[b, :, :n], k0[b, :, :n]) and torch.equal(case.v[b, :, :n], v0[b, :, :n])
        assert torch.equal(case.k[b, :, n:n + m], k0[b, :, n:n + m]) and torch.equal(case.v[b, :, n:n + m], v0[b, :, n:n + m])
        assert torch.equal(case.k[b, :, n + T:], k0[b, :, n + T:])


def test_accept_greedy_reports_malformed_parents_and_argument_errors():
    case = W.make_verify_case(9400, [10], 4, "chain", DEV)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    d = lambda x: torch.tensor(x, dtype=torch.int32, device=DEV)
    path = torch.empty((1, 4), dtype=torch.int32, device=DEV)
    n_acc = torch.empty((1,), dtype=torch.int32, device=DEV)
    bonus = torch.empty((1,), dtype=torch.int32, device=DEV)
    B.sparrow_accept_greedy(ctx, d([[1, 2, 3, 4]]), d([[-1, 0, 7, 2]]), d([[1, 2, 3, 4, 5]]), 4, path, n_acc, bonus)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 3                      # SPARROW_ERR_TREE; node 2 counted as a root
    assert 0 <= int(n_acc[0]) <= 4
    with pytest.raises(B.SparrowError):
        B.sparrow_accept_greedy(ctx, d([[1]]), d([[-1]]), d([[1, 2]]), 0, path, n_acc, bonus)
    with pytest.raises(B.SparrowError):
        B.sparrow_kv_keep_accepted(ctx, case.k, case.v, [case.capacity], path, n_acc, 4)


# ---- temperature 1: rejection sampling over the tree, bit-exact against the oracle --------------

def _sampling_problem(seed, batch, T, vocab, sharp=1.0, same=False):
    """Synthetic distributions (a softmax of seeded normals, sharper for the target), draft tokens
    drawn from the draft rows without replacement among siblings, seeded 32-bit uniforms."""
    rng = np.random.default_rng(seed)
    par = [W.random_tree_parents(seed + 17 * b, 56, T) for b in range(batch)]
    lt = rng.standard_normal((batch, T + 1, vocab)) * 2.0 * sharp
    ld = lt + rng.standard_normal((batch, T + 1, vocab)) * (0.0 if same else 1.0)
    p = np.exp(lt - lt.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
    q = np.exp(ld - ld.max(-1, keepdims=True)); q /= q.sum(-1, keepdims=True)
    p, q = p.astype(np.float32), q.astype(np.float32)
    tok = np.zeros((batch, T), np.int64)
    for b in range(batch):
        for i in range(T):
            row = q[b, par[b][i] + 1].astype(np.float64).copy()
            for j in range(i):
                if par[b][j] == par[b][i]:
                    row[tok[b, j]] = 0.0
            row /= row.sum()
            tok[b, i] = rng.choice(vocab, p=row)
    u_node = rng.integers(0, 1 << 32, size=(batch, T), dtype=np.uint64)
    u_bonus = rng.integers(0, 1 << 32, size=(batch, T + 1), dtype=np.uint64)
    return tok, par, p, q, u_node, u_bonus


def _u32(a):
    return torch.from_numpy(a.astype(np.uint32).view(np.int32).copy()).to(DEV)


@pytest.mark.parametrize("batch,T,vocab,sharp,same", [
    (1, 1, 7, 1.0, False),
    (2, 12, 50, 1.0, False),
    (3, 30, 1000, 0.5, False),          # flat distributions: many rejections per level
    (2, 48, 5000, 2.0, False),          # peaked target
    (1, 25, 151936, 1.0, False),        # a Qwen2-sized vocabulary
    (4, 20, 300, 1.0, True),            # draft = target: everything on the first-child chain is accepted
    (64, 5, 33, 1.0, False),
])
def test_accept_sample_matches_the_oracle(batch, T, vocab, sharp, same):
    tok, par, p, q, u_node, u_bonus = _sampling_problem(9500 + batch + T, batch, T, vocab, sharp, same)
    case = W.make_verify_case(9501, [40] * batch, T, "chain", DEV)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    d = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device=DEV)
    path = torch.full((batch, T), 99, dtype=torch.int32, device=DEV)
    n_acc = torch.full((batch,), 99, dtype=torch.int32, device=DEV)
    bonus = torch.full((batch,), 99, dtype=torch.int32, device=DEV)
    B.sparrow_accept_sample(ctx, d(tok), d(par), torch.from_numpy(p).to(DEV), torch.from_numpy(q).to(DEV),
                            _u32(u_node), _u32(u_bonus), vocab, T, path, n_acc, bonus)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    lengths = []
    for b in range(batch):
        ref_path, ref_bonus = oracle.sample_accept(tok[b], par[b], p[b], q[b], u_node[b], u_bonus[b])
        assert int(n_acc[b]) == len(ref_path)
        assert path[b].tolist() == ref_path + [-1] * (T - len(ref_path))
        assert int(bonus[b]) == ref_bonus
        lengths.append(len(ref_path))
    if same:
        assert min(lengths) >= 1


def test_accept_sample_edge_cases():
    """Zero draft mass on the drafted token, a target row equal to the draft row after a rejection
    (nothing left of the residual: the original row is used), tokens outside the vocabulary."""
    T, V = 3, 4
    par = [[-1, -1, 0]]
    p = np.array([[[0.5, 0.5, 0.0, 0.0]] * (T + 1)], np.float32)
    q = np.array([[[0.5, 0.5, 0.0, 0.0]] * (T + 1)], np.float32)
    case = W.make_verify_case(9502, [40], T, "chain", DEV)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    d = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device=DEV)
    for tok, expect_status in (([[2, 3, 1]], 0), ([[2, 0, 1]], 0), ([[9, -4, 1]], 3)):
        u_node = np.array([[7, 1 << 31, 123456]], np.uint64)
        u_bonus = np.array([[1 << 30, 3 << 30, 5, 77]], np.uint64)
        path = torch.full((1, T), 99, dtype=torch.int32, device=DEV)
        n_acc = torch.full((1,), 99, dtype=torch.int32, device=DEV)
        bonus = torch.full((1,), 99, dtype=torch.int32, device=DEV)
        B.sparrow_accept_sample(ctx, d(tok), d(par), torch.from_numpy(p).to(DEV), torch.from_numpy(q).to(DEV),
                                _u32(u_node), _u32(u_bonus), V, T, path, n_acc, bonus)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == expect_status
        if expect_status == 0:
            ref_path, ref_bonus = oracle.sample_accept(tok[0], par[0], p[0], q[0], u_node[0], u_bonus[0])
            assert path[0, :int(n_acc[0])].tolist() == ref_path and int(bonus[0]) == ref_bonus
        else:
            assert int(n_acc[0]) == 0 and 0 <= int(bonus[0]) < V
    with pytest.raises(B.SparrowError):
        B.sparrow_accept_sample(ctx, d([[0]]), d([[-1]]), torch.from_numpy(p).to(DEV), torch.from_numpy(q).to(DEV),
                                _u32(np.zeros((1, 1), np.uint64)), _u32(np.zeros((1, 2), np.uint64)), 0, 1, path, n_acc, bonus)
