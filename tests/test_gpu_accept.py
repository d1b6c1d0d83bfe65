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
