"""The entry point for callers that cannot allocate device memory (hosts that own the whole
memory pool, loops that cannot afford cudaMalloc): sparrow_verify_attn_static() keeps its scratch
in a fixed array inside the library.  It must agree with the ordinary, context-based entry point
and with the CPU oracle on the same inputs -- on calls in a row, since all calls share that one
array -- and must refuse work that does not fit the array.  Collected last on purpose (file name)."""
import pytest
import torch

from paper_2602_15318_b200 import binding as B
from paper_2602_15318_b200 import workloads as W

from gpu_util import TOL_LSE, TOL_OUT, check, oracle_verify

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _layout(case):
    k = case.k
    return B.Layout(k.shape[0], W.HQ, k.shape[1], k.shape[3], k.shape[2], W.SCALE, k.stride(0), k.stride(1))


def _with_context(case):
    ctx = B.Context.for_cache(case.k, W.SCALE)
    out = torch.full_like(case.q, float("nan"))
    lse = torch.full((case.B, W.HQ, case.T), float("nan"), dtype=torch.float32, device=DEV)
    B.sparrow_verify_attn(ctx, case.q, case.k, case.v, case.kv_len, case.parents, case.T, out, lse)
    torch.cuda.synchronize()
    return out, lse


def _static(case):
    out = torch.full_like(case.q, float("nan"))
    lse = torch.full((case.B, W.HQ, case.T), float("nan"), dtype=torch.float32, device=DEV)
    B.sparrow_verify_attn_static(_layout(case), case.q, case.k, case.v, case.kv_len, case.parents, case.T, out, lse)
    torch.cuda.synchronize()
    return out, lse


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    torch.cuda.set_device(0)
    first = W.make_verify_case(9001, [5000], 16, "chain", DEV)            # many pieces per unit
    second = W.make_verify_case(9002, [700, 2300], 24, "random", DEV)     # other layout, two row blocks
    third = W.make_verify_case(9004, [1500], 64, "random", DEV)           # the largest draft block: two row groups
    oracle_results = {}
    for case in (first, second, third, first):
        ref_out, ref_lse = _with_context(case)
        out, lse = _static(case)
        assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
        assert float((out.float() - ref_out.float()).abs().max()) <= TOL_OUT
        assert float((lse - ref_lse).abs().max()) <= TOL_LSE
        # and against the oracle: a defect shared by the two entry points must not pass
        if id(case) not in oracle_results:
            oracle_results[id(case)] = oracle_verify(case)
        check(out, lse, *oracle_results[id(case)])


def test_static_entry_point_refuses_what_does_not_fit():
    torch.cuda.set_device(0)
    big = W.make_verify_case(9003, [100] * 32, 64, "random", DEV)         # 256 work items of 70 KB
    out = torch.empty_like(big.q)
    lse = torch.empty((big.B, W.HQ, big.T), dtype=torch.float32, device=DEV)
    with pytest.raises(B.SparrowError) as e:
        B.sparrow_verify_attn_static(_layout(big), big.q, big.k, big.v, big.kv_len, big.parents, big.T, out, lse)
    assert e.value.status == 5                                             # SPARROW_ERR_WORKSPACE


def test_static_entry_point_checks_arguments_before_touching_the_gpu():
    torch.cuda.set_device(0)
    case = W.make_verify_case(9005, [200], 4, "chain", DEV)
    out = torch.empty_like(case.q)
    lse = torch.empty((1, W.HQ, 4), dtype=torch.float32, device=DEV)
    for kw, status in [(dict(T=0), 2), (dict(T=65), 2), (dict(kv_len=[-1]), 2), (dict(kv_len=[201]), 2),
                       (dict(q=None), 1), (dict(parents=None), 1)]:
        args = dict(q=case.q, kv_len=case.kv_len, parents=case.parents, T=4)
        args.update(kw)
        with pytest.raises(B.SparrowError) as e:
            B.sparrow_verify_attn_static(_layout(case), args["q"], case.k, case.v, args["kv_len"], args["parents"],
                                         args["T"], out, lse)
        assert e.value.status == status
