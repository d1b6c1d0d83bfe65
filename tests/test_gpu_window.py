"""GPU parity of the text-anchored window mode on a compacted cache: sparrow_compact_anchors()
once, then sparrow_verify_attn_window() -- a contiguous stream for the tensor-core kernel with a
per-query lower bound -- against the anchored oracle on the full-length cache."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_15318_b200 import binding as B
from paper_2602_15318_b200 import workloads as W

from gpu_util import anchor_case, check

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _compact(ac, ctx):
    cap = ac.n_anchor + 3
    kc = torch.zeros((ac.B, W.HKV, cap, W.D), dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    B.sparrow_compact_anchors(ctx, ac.k, ac.v, ac.anchor_idx, ac.n_anchor, kc, vc, cap, 0)
    return kc, vc


def _run(ac, parents, T_tree, T_new, bounds="device", give_min=True, policy=None):
    """Compacts, derives the window bounds (on the device or on the host), runs the windowed call;
    returns (out, lse, oracle out, oracle lse)."""
    ctx = B.Context.for_cache(ac.k, W.SCALE)
    kc, vc = _compact(ac, ctx)
    cctx = B.Context.for_cache(kc, W.SCALE)
    if policy is not None:
        cctx.set_plan_policy(policy)
    q = ac.q[:, T_tree - T_new:].contiguous()
    host = [B.sparrow_window_first_visible(ac.anchor_idx[b].tolist(), ac.window, T_tree, T_new) for b in range(ac.B)]
    if bounds == "device":
        first = torch.full((ac.B, T_new), -7, dtype=torch.int32, device=DEV)
        B.sparrow_window_first_visible_device(ctx, ac.anchor_idx, ac.n_anchor, ac.window, T_tree, T_new, first)
        torch.cuda.synchronize()
        assert first.cpu().tolist() == [h[0] for h in host]               # bit-exact against the host helper
    elif bounds == "host":
        first = torch.tensor([h[0] for h in host], dtype=torch.int32, device=DEV)
    else:
        first = None
    out = torch.full_like(q, float("nan"))
    lse = torch.full((ac.B, W.HQ, T_new), float("nan"), dtype=torch.float32, device=DEV)
    B.sparrow_verify_attn_window(cctx, q, kc, vc, [ac.n_anchor - T_tree] * ac.B, parents, T_tree, T_new, first,
                                 [h[1] for h in host] if (give_min and first is not None) else None, out, lse)
    torch.cuda.synchronize()
    assert cctx.last_device_status() == 0 and ctx.last_device_status() == 0
    ref = oracle.anchor_attn_tree(W.bf16_bits(q), W.bf16_bits(ac.k), W.bf16_bits(ac.v), ac.anchor_idx.cpu().numpy(),
                                  ac.window, parents.cpu().numpy(), W.SCALE)
    return out, lse, ref[0], ref[1]


def _chain(T, batch):
    return torch.tensor([W.chain_parents(T)] * batch, dtype=torch.int32, device=DEV)


def _trees(seed, T, batch):
    return torch.tensor([W.random_tree_parents(seed + 31 * b, 99, T) for b in range(batch)], dtype=torch.int32, device=DEV)


def test_config4_on_the_compacted_cache():
    """The anchored configuration (448 text anchors, window 1024, 8 chain tokens): every anchor is
    inside every query's window, the bounds are all zero."""
    ac = W.make_config(3, DEV)
    out, lse, ref_out, ref_lse = _run(ac, _chain(8, 1), 8, 8)
    check(out, lse, ref_out, ref_lse)
    plain = oracle.anchor_attn(W.bf16_bits(ac.q), W.bf16_bits(ac.k), W.bf16_bits(ac.v), ac.anchor_idx.cpu().numpy(),
                               ac.window, W.SCALE)
    check(out, lse, *plain)                                               # and it is the chain mode of Eq. 2


@pytest.mark.parametrize("seq_len,spans,window,T_tree,T_new,batch,bounds", [
    (30000, [[100, 19900]], 3000, 24, 8, 1, "device"),       # ~10k text anchors, the window keeps the last ~3000
    (30000, [[100, 19900]], 3000, 24, 24, 1, "host"),
    (6000, [[0, 700], [2000, 2600]], 1500, 40, 10, 2, "device"),
    (3000, [[40, 2600]], 130, 10, 10, 2, "device"),          # the cut falls inside the last tile, next to the tree
    (3000, [[40, 2600]], 0, 10, 3, 1, "none"),               # no window, no bounds array at all
    (900, [[0, 850]], 20, 64, 64, 1, "host"),                # largest tree; the window is shorter than the tree itself
    (5000, [[10, 400]], 4000, 19, 19, 3, "device"),          # two row blocks, bounds differ from row to row
])
def test_window_on_compacted_cache_matches_anchored_oracle(seq_len, spans, window, T_tree, T_new, batch, bounds):
    ac = anchor_case(5100 + T_tree + window, seq_len, spans, window, T_tree, batch, DEV)
    out, lse, ref_out, ref_lse = _run(ac, _trees(5200 + T_tree, T_tree, batch), T_tree, T_new, bounds=bounds)
    check(out, lse, ref_out, ref_lse)


@pytest.mark.parametrize("policy", [B.PLAN_LATENCY, B.PLAN_THROUGHPUT])
def test_window_bounds_that_differ_per_query_and_explicit_anchor_gaps(policy):
    """An explicit anchor list with irregular gaps: consecutive queries cut the list at different
    places, some of them several tiles apart; with and without the host-side lower bound."""
    rng = np.random.default_rng(11)
    T = 12
    text = np.sort(rng.choice(50000, size=4000, replace=False))
    rows = 50000 + np.arange(0, 40 * T, 40)                               # draft rows far apart: bounds 40 positions apart
    idx = np.concatenate([text, rows]).tolist()
    ac = W.make_anchor_case(5300, idx, 9000, T, 1, DEV)
    par = _trees(5301, T, 1)
    for give_min in (True, False):
        out, lse, ref_out, ref_lse = _run(ac, par, T, T, bounds="device", give_min=give_min, policy=policy)
        check(out, lse, ref_out, ref_lse)


def test_window_bound_left_of_the_streamed_keys_is_reported():
    ac = W.make_anchor_case(5400, list(range(3000)) + list(range(3000, 3006)), 900, 6, 1, DEV)
    ctx = B.Context.for_cache(ac.k, W.SCALE)
    kc, vc = _compact(ac, ctx)
    cctx = B.Context.for_cache(kc, W.SCALE)
    first, lowest = B.sparrow_window_first_visible(ac.anchor_idx[0].tolist(), ac.window, 6, 6)
    assert lowest >= 256
    dev_first = torch.tensor([first], dtype=torch.int32, device=DEV)
    dev_first[0, 2] = 5                                                   # contradicts the host-side minimum
    out = torch.empty_like(ac.q)
    lse = torch.empty((1, W.HQ, 6), dtype=torch.float32, device=DEV)
    B.sparrow_verify_attn_window(cctx, ac.q, kc, vc, [ac.n_anchor - 6], _chain(6, 1), 6, 6, dev_first, [lowest], out, lse)
    torch.cuda.synchronize()
    assert cctx.last_device_status() == 4                                 # SPARROW_ERR_ANCHOR
    assert torch.isfinite(out.float()).all()
    with pytest.raises(B.SparrowError):
        B.sparrow_verify_attn_window(cctx, ac.q, kc, vc, [ac.n_anchor - 6], _chain(6, 1), 6, 7, dev_first, None, out, lse)
    with pytest.raises(B.SparrowError):
        B.sparrow_verify_attn_window(cctx, ac.q, kc, vc, [ac.n_anchor - 6], _chain(6, 1), 6, 6, dev_first,
                                     [ac.n_anchor], out, lse)            # minimum beyond the prefix
