"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances (bf16 inputs, fp32 accumulation): max |d out| <= 1e-2, max |d lse| <= 1e-3; masks and
indices bit-exact.  Every case is compared element by element, the five full-size configurations
included (three whole layers of the batched step; its 28-layer sweep checks sampled rows of every
layer on top of that).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_15318_b200 import binding as B
from paper_2602_15318_b200 import workloads as W

from gpu_util import (anchor_case, check, compare, oracle_anchor, oracle_verify, run_anchor,
                      run_verify, sample_rows)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


# ---- verification mode: small shapes spanning several tiles and ragged tails ---------------

@pytest.mark.parametrize("kv_len,T,tree", [
    ([300], 5, "chain"),
    ([1], 1, "chain"),
    ([0], 7, "chain"),             # no prefix at all: only the draft block
    ([0], 1, "chain"),             # a single key
    ([63], 3, "forest"),
    ([64], 8, "random"),
    ([129], 19, "random"),         # 133 packed rows: two row groups
    ([1000], 64, "random"),        # 448 packed rows
    ([4099], 16, "chain"),
    ([1, 130, 517], 9, "random"),  # ragged batch
    ([777, 5, 2048, 64], 32, "random"),
])
def test_verify_small(kv_len, T, tree):
    case = W.make_verify_case(1234 + T + len(kv_len), kv_len, T, tree, DEV)
    out, lse, _ = run_verify(case)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


@pytest.mark.parametrize("T", [17, 18, 19, 35, 36, 37, 54, 55, 63])
@pytest.mark.parametrize("policy", [B.PLAN_LATENCY, B.PLAN_THROUGHPUT])
def test_verify_row_block_boundaries(T, policy):
    """Draft blocks around the 18-token row blocks and 36-token row groups, random trees, a key
    count that ends inside a tile; one wave of pieces and a few long ones."""
    case = W.make_verify_case(3000 + T, [2300 - T, 700], T, "random", DEV)
    out, lse, _ = run_verify(case, policy=policy)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


@pytest.mark.parametrize("n_keys", [127, 128, 129, 255, 256, 257, 384])
def test_verify_key_counts_around_tile_boundaries(n_keys):
    T = 6
    case = W.make_verify_case(3100 + n_keys, [n_keys - T], T, "chain", DEV)
    out, lse, _ = run_verify(case)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


def test_verify_largest_batch():
    lens = [(37 * i) % 300 for i in range(64)]
    case = W.make_verify_case(3200, lens, 5, "random", DEV)
    out, lse, _ = run_verify(case)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


def test_verify_capacity_larger_than_used_and_garbage_tail():
    """Rows past kv_len+T may hold anything, NaN and Inf patterns included."""
    case = W.make_verify_case(77, [200, 333], 6, "random", DEV, capacity=700)
    for b, n in enumerate(case.kv_len):
        case.k[b, :, n + case.T:, :] = float("nan")
        case.v[b, :, n + case.T:, :] = float("inf")
        case.v[b, :, n + case.T + 3:, :] = float("nan")
    out, lse, _ = run_verify(case)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


def test_verify_strided_cache_view():
    """A cache whose head stride is larger than capacity*128 (a view into a bigger buffer)."""
    big = W.make_verify_case(78, [150], 4, "chain", DEV, capacity=400)
    kview, vview = big.k[:, :, :200, :], big.v[:, :, :200, :]
    ctx = B.Context(1, 200, kview.stride(0), kview.stride(1), W.SCALE)
    out = torch.empty_like(big.q)
    lse = torch.empty((1, W.HQ, 4), dtype=torch.float32, device=DEV)
    B.sparrow_verify_attn(ctx, big.q, kview, vview, big.kv_len, big.parents, 4, out, lse)
    torch.cuda.synchronize()
    ref_out, ref_lse = oracle_verify(big)
    check(out, lse, ref_out, ref_lse)


def test_verify_deterministic_and_context_reuse():
    case = W.make_verify_case(79, [3000, 1500], 12, "random", DEV)
    out1, lse1, ctx = run_verify(case)
    out2, lse2, _ = run_verify(case, ctx)
    assert torch.equal(out1.view(torch.int16), out2.view(torch.int16))
    assert torch.equal(lse1, lse2)
    other = W.make_verify_case(80, [100, 2900], 3, "chain", DEV, capacity=case.capacity)
    out3, lse3, _ = run_verify(other, ctx)          # different T and lengths, same context
    ref_out, ref_lse = oracle_verify(other)
    check(out3, lse3, ref_out, ref_lse)


def test_verify_on_side_stream():
    case = W.make_verify_case(81, [2000], 8, "chain", DEV)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    out = torch.empty_like(case.q)
    lse = torch.empty((1, W.HQ, 8), dtype=torch.float32, device=DEV)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        B.sparrow_verify_attn(ctx, case.q, case.k, case.v, case.kv_len, case.parents, 8, out, lse)
    s.synchronize()
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


# ---- other head geometries (query heads per KV head from 1 to 16) ----------------------------------

@pytest.mark.parametrize("hq,hkv,kv_len,T,tree,policy", [
    (32, 8, [3000, 700], 12, "random", B.PLAN_LATENCY),        # group 4: 32 tokens per row block
    (32, 8, [2000], 40, "random", B.PLAN_THROUGHPUT),          # group 4, two row blocks
    (32, 4, [2500], 16, "chain", B.PLAN_BALANCED),             # group 8: 16 tokens per block, no padding rows
    (32, 4, [1500, 90], 33, "random", B.PLAN_LATENCY),         # group 8: three blocks -> two row groups
    (8, 8, [1800], 64, "random", B.PLAN_LATENCY),              # multi-head attention: one head per KV head
    (16, 1, [4000], 9, "random", B.PLAN_THROUGHPUT),           # multi-query attention, group 16: 8 tokens per block
    (16, 1, [600], 64, "random", B.PLAN_LATENCY),              # group 16: eight blocks, four row groups
    (12, 4, [1000, 1000, 5], 50, "random", B.PLAN_BALANCED),   # group 3: 42 tokens per block
    (10, 2, [777], 26, "chain", B.PLAN_LATENCY),               # group 5: 25 tokens per block, 3 rows of padding
])
def test_verify_other_gqa_ratios(hq, hkv, kv_len, T, tree, policy):
    case = W.make_verify_case(3300 + hq + T, kv_len, T, tree, DEV, hq=hq, hkv=hkv)
    out, lse, _ = run_verify(case, policy=policy)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


def test_anchored_modes_with_another_gqa_ratio():
    """Group 4 (32 / 8 heads): the gather kernel, and the compacted cache with a cutting window."""
    hq, hkv, T = 32, 8, 10
    idx = oracle.anchor_idx(6000, [[50, 4000]], 1200, T).tolist()
    base = W.make_verify_case(3400, [idx[-1] + 1 - T], T, "chain", DEV, hq=hq, hkv=hkv)       # tensors only
    anchor = torch.tensor([idx], dtype=torch.int32, device=DEV)
    parents = torch.tensor([W.random_tree_parents(3401, 99, T)], dtype=torch.int32, device=DEV)
    ctx = B.Context.for_cache(base.k, W.SCALE, n_q_heads=hq)
    ref = oracle.anchor_attn_tree(W.bf16_bits(base.q), W.bf16_bits(base.k), W.bf16_bits(base.v), anchor.cpu().numpy(), 1200,
                                  parents.cpu().numpy(), W.SCALE)
    out = torch.full_like(base.q, float("nan"))
    lse = torch.full((1, hq, T), float("nan"), dtype=torch.float32, device=DEV)
    B.sparrow_anchor_attn_tree(ctx, base.q, base.k, base.v, anchor, len(idx), 1200, parents, T, T, out, lse)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    check(out, lse, *ref)
    kc = torch.zeros((1, hkv, len(idx), W.D), dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    B.sparrow_compact_anchors(ctx, base.k, base.v, anchor, len(idx), kc, vc, len(idx), 0)
    first = torch.empty((1, T), dtype=torch.int32, device=DEV)
    B.sparrow_window_first_visible_device(ctx, anchor, len(idx), 1200, T, T, first)
    cctx = B.Context.for_cache(kc, W.SCALE, n_q_heads=hq)
    out2 = torch.full_like(base.q, float("nan"))
    lse2 = torch.full((1, hq, T), float("nan"), dtype=torch.float32, device=DEV)
    B.sparrow_verify_attn_window(cctx, base.q, kc, vc, [len(idx) - T], parents, T, T, first, None, out2, lse2)
    torch.cuda.synchronize()
    assert cctx.last_device_status() == 0
    check(out2, lse2, *ref)


# ---- masks and indices: bit-exact -----------------------------------------------------------

def test_device_ancestor_masks_bit_exact():
    ctx = B.Context(1, 128, 4 * 128 * 128, 128 * 128, W.SCALE)
    trees = [W.chain_parents(64), [-1] * 64, [-1], [-1, 0, 0, 2, 1, 1, 5]]
    trees += [W.random_tree_parents(s, 4, T) for s, T in [(1, 64), (2, 48), (3, 30), (4, 25), (5, 2)]]
    for par in trees:
        dev = torch.tensor(par, dtype=torch.int32, device=DEV)
        masks = B.sparrow_debug_ancestor_masks_device(ctx, dev, len(par))
        torch.cuda.synchronize()
        got = masks.cpu().numpy().view(np.uint64)
        assert np.array_equal(got, oracle.ancestor_masks(np.array(par, np.int32)))
    assert ctx.last_device_status() == 0


def test_device_reports_malformed_parents_without_faulting():
    ctx = B.Context(1, 128, 4 * 128 * 128, 128 * 128, W.SCALE)
    dev = torch.tensor([-1, 0, 5, 1, -3, 2], dtype=torch.int32, device=DEV)   # 5 >= 2, -3 < -1
    masks = B.sparrow_debug_ancestor_masks_device(ctx, dev, 6)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 3            # SPARROW_ERR_TREE, sticky until read
    assert ctx.last_device_status() == 0
    got = masks.cpu().numpy().view(np.uint64)
    assert int(got[2]) == 0b100 and int(got[4]) == 0b10000        # bad parent treated as root


def test_masking_is_exact_under_one_hot_values():
    """With V = one-hot rows the output row is the softmax weight vector itself: entries of
    invisible draft keys must be exactly zero, visible ones positive."""
    T, kv_len = 16, 40
    case = W.make_verify_case(90, [kv_len], T, "random", DEV, capacity=128)
    case.v.zero_()
    n = kv_len + T
    case.v[0, :, torch.arange(n), torch.arange(n)] = 1.0
    out, lse, _ = run_verify(case)
    anc = oracle.ancestor_masks(case.parents[0].cpu().numpy())
    vis = oracle.verify_visibility(kv_len, anc).astype(bool)           # [T, n]
    w = out[0].float().cpu().numpy()                                   # [T, Hq, 128]
    for t in range(T):
        assert np.all(w[t][:, :n][:, ~vis[t]] == 0.0)
        assert np.all(w[t][:, :n][:, vis[t]] >= 0.0)
        assert np.all(w[t][:, n:] == 0.0)
        np.testing.assert_allclose(w[t].sum(axis=1), 1.0, atol=2e-2)


# ---- anchored mode ---------------------------------------------------------------------------

@pytest.mark.parametrize("seq_len,spans,window,T,batch", [
    (300, [[10, 250]], 0, 4, 1),
    (500, [[0, 100], [200, 420]], 64, 8, 2),
    (1000, [], 0, 3, 1),                  # nothing visual: plain causal over everything
    (2000, [[5, 1990]], 100, 16, 1),
    (90, [[0, 90]], 0, 5, 1),             # only the draft block remains
])
def test_anchor_small(seq_len, spans, window, T, batch):
    case = anchor_case(4321 + T, seq_len, spans, window, T, batch, DEV)
    assert case.anchor_idx[0].tolist() == B.sparrow_build_anchor_idx(seq_len, spans, window, T)
    out, lse, _ = run_anchor(case)
    ref_out, ref_lse = oracle_anchor(case)
    check(out, lse, ref_out, ref_lse)


def test_anchor_window_drops_old_anchors():
    """An explicit anchor list where the per-query window bound cuts inside the list."""
    T = 3
    idx = list(range(0, 400, 3)) + [1000, 1001, 1002]
    case = anchor_case(55, 1000, [], 0, T, 1, DEV)
    case.anchor_idx = torch.tensor([idx], dtype=torch.int32, device=DEV)
    case.n_anchor = len(idx)
    case.window = 700
    out, lse, _ = run_anchor(case)
    ref_out, ref_lse = oracle_anchor(case)
    check(out, lse, ref_out, ref_lse)


def test_anchor_out_of_range_index_is_reported_not_read():
    case = anchor_case(56, 200, [[20, 150]], 0, 4, 1, DEV)
    bad = case.anchor_idx.clone()
    bad[0, 3] = 10 ** 6
    case.anchor_idx = bad
    ctx = B.Context.for_cache(case.k, W.SCALE)
    out = torch.empty_like(case.q)
    lse = torch.empty((1, W.HQ, 4), dtype=torch.float32, device=DEV)
    B.sparrow_anchor_attn(ctx, case.q, case.k, case.v, case.anchor_idx, case.n_anchor, 0, 4, out, lse)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 4
    assert torch.isfinite(out.float()).all()


# ---- the five configurations at full size ---------------------------------------------------

def test_config1_full():
    case = W.make_config(0, DEV)
    out, lse, _ = run_verify(case)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


POLICIES = [B.PLAN_LATENCY, B.PLAN_BALANCED, B.PLAN_THROUGHPUT]


def _full_rows_under_every_policy(config_index):
    """Every (token, head) row of the configuration against the oracle (computed once), with the
    key range cut under each planner policy."""
    case = W.make_config(config_index, DEV)
    ref_out, ref_lse = oracle_verify(case)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    for policy in POLICIES:
        out, lse, _ = run_verify(case, ctx, policy=policy)
        check(out, lse, ref_out, ref_lse)


def test_config2_every_row_every_policy():
    _full_rows_under_every_policy(1)


def test_config3_every_row_every_policy():
    _full_rows_under_every_policy(2)


def test_config4_full():
    case = W.make_config(3, DEV)
    assert case.n_anchor == 456
    out, lse, _ = run_anchor(case)
    ref_out, ref_lse = oracle_anchor(case)
    check(out, lse, ref_out, ref_lse)


@pytest.mark.parametrize("layer,policy", [(0, B.PLAN_BALANCED), (13, B.PLAN_THROUGHPUT), (27, B.PLAN_LATENCY)])
def test_config5_layer_every_row(layer, policy):
    """One whole layer of the batched step: all 8 x 32 x 28 rows against the oracle."""
    case = W.make_config(4, DEV, layer=layer)
    out, lse, _ = run_verify(case, policy=policy)
    ref_out, ref_lse = oracle_verify(case)
    check(out, lse, ref_out, ref_lse)


def test_config5_every_layer_sampled_rows():
    """All 28 per-layer caches of the batched step, one after the other (generate, run, check a few
    rows of every sequence against the oracle), the planner policy changing from layer to layer."""
    ctx = None
    for layer in range(28):
        case = W.make_config(4, DEV, layer=layer)
        ctx = ctx or B.Context.for_cache(case.k, W.SCALE)
        out, lse, _ = run_verify(case, ctx, policy=POLICIES[layer % 3])
        rows = sample_rows(500 + layer, 8, case.T, 12)
        ref_out, ref_lse = oracle_verify(case, rows)
        check(out, lse, ref_out, ref_lse, rows)
        del case, out, lse
        torch.cuda.empty_cache()


# ---- host-buffer entry point and argument errors --------------------------------------------

def test_verify_step_host_matches_device_call():
    case = W.make_verify_case(91, [900, 411], 10, "random", DEV, capacity=1024)
    ref_out, ref_lse = oracle_verify(case)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    T = case.T
    q_h = case.q.cpu().pin_memory()
    k_new = torch.stack([case.k[b, :, n:n + T, :] for b, n in enumerate(case.kv_len)]).cpu().pin_memory()
    v_new = torch.stack([case.v[b, :, n:n + T, :] for b, n in enumerate(case.kv_len)]).cpu().pin_memory()
    for b, n in enumerate(case.kv_len):            # the call must write the draft rows itself
        case.k[b, :, n:n + T, :] = 0
        case.v[b, :, n:n + T, :] = 0
    out_h = torch.empty_like(q_h).pin_memory()
    lse_h = torch.empty((2, W.HQ, T), dtype=torch.float32).pin_memory()
    B.sparrow_verify_step_host(ctx, q_h, k_new, v_new, case.k, case.v, case.kv_len,
                               case.parents.cpu(), T, out_h, lse_h)
    check(out_h, lse_h, ref_out, ref_lse)


def test_verify_step_host_pinned_buffers_twice():
    """All six host buffers page-locked: the kernels read and write them over the host link.  The
    second step reuses the same host buffers with other contents, so a stale cached line would show."""
    ctx = None
    bufs = None
    for seed, lens in [(93, [1500, 700]), (94, [1490, 333])]:
        case = W.make_verify_case(seed, lens, 12, "random", DEV, capacity=2048)
        ref_out, ref_lse = oracle_verify(case)
        T = case.T
        if ctx is None:
            ctx = B.Context.for_cache(case.k, W.SCALE)
            bufs = dict(q=torch.empty(case.q.shape, dtype=case.q.dtype).pin_memory(),
                        k=torch.empty((2, W.HKV, T, W.D), dtype=case.k.dtype).pin_memory(),
                        v=torch.empty((2, W.HKV, T, W.D), dtype=case.k.dtype).pin_memory(),
                        par=torch.empty((2, T), dtype=torch.int32).pin_memory(),
                        out=torch.empty(case.q.shape, dtype=case.q.dtype).pin_memory(),
                        lse=torch.empty((2, W.HQ, T), dtype=torch.float32).pin_memory())
        bufs["q"].copy_(case.q)
        bufs["k"].copy_(torch.stack([case.k[b, :, n:n + T, :] for b, n in enumerate(case.kv_len)]))
        bufs["v"].copy_(torch.stack([case.v[b, :, n:n + T, :] for b, n in enumerate(case.kv_len)]))
        bufs["par"].copy_(case.parents)
        bufs["out"].zero_(); bufs["lse"].zero_()
        torch.cuda.synchronize()
        for b, n in enumerate(case.kv_len):
            case.k[b, :, n:n + T, :] = 0
            case.v[b, :, n:n + T, :] = 0
        n0 = ctx.launch_count()
        B.sparrow_verify_step_host(ctx, bufs["q"], bufs["k"], bufs["v"], case.k, case.v, case.kv_len,
                                   bufs["par"], T, bufs["out"], bufs["lse"])
        assert ctx.launch_count() - n0 == 2          # the ingest kernel and the attention kernel
        check(bufs["out"], bufs["lse"], ref_out, ref_lse)
        for b, n in enumerate(case.kv_len):          # the new rows reached the cache bit for bit
            assert torch.equal(case.k[b, :, n:n + T, :].cpu(), bufs["k"][b])
            assert torch.equal(case.v[b, :, n:n + T, :].cpu(), bufs["v"][b])


def test_verify_step_host_pinned_ragged_batch_tree():
    """The page-locked route on a ragged batch of 8 with a 32-node tree (two row blocks per tile,
    results stored straight into host memory by the finishers of every sequence)."""
    lens = [1900, 37, 1024, 0, 777, 1500, 129, 640]
    case = W.make_verify_case(95, lens, 32, "random", DEV, capacity=2048)
    ref_out, ref_lse = oracle_verify(case)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    T, nb = case.T, len(lens)
    q_h = case.q.cpu().pin_memory()
    k_new = torch.stack([case.k[b, :, n:n + T, :] for b, n in enumerate(case.kv_len)]).cpu().pin_memory()
    v_new = torch.stack([case.v[b, :, n:n + T, :] for b, n in enumerate(case.kv_len)]).cpu().pin_memory()
    par_h = case.parents.cpu().pin_memory()
    for b, n in enumerate(case.kv_len):
        case.k[b, :, n:n + T, :] = float("nan")
        case.v[b, :, n:n + T, :] = float("nan")
    out_h = torch.full(q_h.shape, float("nan"), dtype=q_h.dtype).pin_memory()
    lse_h = torch.full((nb, W.HQ, T), float("nan"), dtype=torch.float32).pin_memory()
    B.sparrow_verify_step_host(ctx, q_h, k_new, v_new, case.k, case.v, case.kv_len, par_h, T, out_h, lse_h)
    assert ctx.last_device_status() == 0
    check(out_h, lse_h, ref_out, ref_lse)


def test_argument_errors_launch_nothing():
    case = W.make_verify_case(92, [100], 4, "chain", DEV)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    out = torch.empty_like(case.q)
    lse = torch.empty((1, W.HQ, 4), dtype=torch.float32, device=DEV)
    n0 = ctx.launch_count()
    for kw, status in [(dict(T=0), 2), (dict(T=65), 2), (dict(kv_len=[-1]), 2), (dict(kv_len=[101]), 2),
                       (dict(q=None), 1), (dict(parents=None), 1)]:
        args = dict(q=case.q, kv_len=case.kv_len, parents=case.parents, T=4)
        args.update(kw)
        with pytest.raises(B.SparrowError) as e:
            B.sparrow_verify_attn(ctx, args["q"], case.k, case.v, args["kv_len"], args["parents"],
                                  args["T"], out, lse)
        assert e.value.status == status
    with pytest.raises(B.SparrowError) as e:
        B.sparrow_anchor_attn(ctx, case.q, case.k, case.v, case.parents, 2, 0, 4, out, lse)
    assert e.value.status == 4                      # n_anchor < T
    bare = B.Context.for_cache(case.k, W.SCALE, allocate_workspace=False)
    with pytest.raises(B.SparrowError) as e:
        B.sparrow_verify_attn(bare, case.q, case.k, case.v, case.kv_len, case.parents, 4, out, lse)
    assert e.value.status == 5
    with pytest.raises(B.SparrowError):
        B.Context(1, 100, 51200, 12800, W.SCALE, n_q_heads=30)       # not a multiple of the 4 KV heads
    with pytest.raises(B.SparrowError):
        B.Context(1, 100, 51200, 12800, W.SCALE, n_q_heads=68)       # 17 query heads per KV head: more than 16
    with pytest.raises(B.SparrowError):
        B.Context(1, 100, 51200, 12800, W.SCALE, head_dim=64, n_q_heads=28)
    assert ctx.launch_count() == n0


# ---- anchored mode with tree-structured draft tokens ---------------------------------------------

def _run_anchor_tree(ac, parents, T_tree, T_new, ctx=None):
    ctx = ctx or B.Context.for_cache(ac.k, W.SCALE)
    q = ac.q[:, T_tree - T_new:].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((ac.B, W.HQ, T_new), float("nan"), dtype=torch.float32, device=DEV)
    B.sparrow_anchor_attn_tree(ctx, q, ac.k, ac.v, ac.anchor_idx, ac.n_anchor, ac.window, parents, T_tree, T_new,
                               out, lse)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    ref_out, ref_lse = oracle.anchor_attn_tree(W.bf16_bits(q), W.bf16_bits(ac.k), W.bf16_bits(ac.v),
                                               ac.anchor_idx.cpu().numpy(), ac.window, parents.cpu().numpy(), W.SCALE)
    return out, lse, ref_out, ref_lse


@pytest.mark.parametrize("seq_len,spans,window,T_tree,T_new,batch", [
    (1500, [[32, 1300]], 0, 12, 12, 1),          # whole tree, no window
    (1500, [[32, 1300]], 128, 12, 5, 2),         # only the nodes of the latest step are queries
    (5000, [[100, 4200]], 600, 40, 8, 1),        # many text anchors: several pieces, tree inside the last tile
    (900, [[0, 850]], 0, 64, 64, 1),             # largest tree: four row blocks' worth of query rows
    (300, [], 0, 9, 1, 3),                       # no visual span, a single query node
])
def test_anchor_tree_small(seq_len, spans, window, T_tree, T_new, batch):
    ac = anchor_case(4100 + T_tree, seq_len, spans, window, T_tree, batch, DEV)
    parents = torch.tensor([W.random_tree_parents(4200 + 31 * b + T_tree, 99, T_tree) for b in range(batch)],
                           dtype=torch.int32, device=DEV)
    out, lse, ref_out, ref_lse = _run_anchor_tree(ac, parents, T_tree, T_new)
    check(out, lse, ref_out, ref_lse)


def test_anchor_tree_with_chain_parents_is_the_chain_mode():
    ac = anchor_case(4300, 2000, [[64, 1700]], 512, 10, 2, DEV)
    chain = torch.tensor([list(range(-1, 9))] * 2, dtype=torch.int32, device=DEV)
    ctx = B.Context.for_cache(ac.k, W.SCALE)
    out_c, lse_c, _ = run_anchor(ac, ctx)
    out_t, lse_t, _, _ = _run_anchor_tree(ac, chain, 10, 10, ctx)
    assert torch.equal(out_c, out_t) and torch.equal(lse_c, lse_t)


def test_anchor_tree_argument_errors():
    ac = anchor_case(4400, 500, [[10, 400]], 0, 8, 1, DEV)
    par = torch.tensor([[-1, 0, 0, 1, 1, 2, 3, 3]], dtype=torch.int32, device=DEV)
    ctx = B.Context.for_cache(ac.k, W.SCALE)
    out = torch.empty_like(ac.q); lse = torch.empty((1, W.HQ, 8), dtype=torch.float32, device=DEV)
    n0 = ctx.launch_count()
    for T_tree, T_new, n_anchor in ((8, 9, ac.n_anchor), (0, 1, ac.n_anchor), (65, 8, ac.n_anchor), (8, 8, 5)):
        with pytest.raises(B.SparrowError):
            B.sparrow_anchor_attn_tree(ctx, ac.q, ac.k, ac.v, ac.anchor_idx, n_anchor, 0, par, T_tree, T_new, out, lse)
    assert ctx.launch_count() == n0
    bad = torch.tensor([[-1, 0, 5, 1, 1, 2, 3, 3]], dtype=torch.int32, device=DEV)      # parents[2] = 5 > 2
    B.sparrow_anchor_attn_tree(ctx, ac.q, ac.k, ac.v, ac.anchor_idx, ac.n_anchor, 0, bad, 8, 8, out, lse)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 3          # SPARROW_ERR_TREE, reported, nothing read out of bounds
    assert torch.isfinite(out.float()).all()


# ---- row movers: append of the draft rows, compaction of the anchored rows -------------------

def test_kv_append_is_a_bit_exact_copy_into_the_right_rows():
    case = W.make_verify_case(4500, [300, 77], 6, "chain", DEV, capacity=400)
    ctx = B.Context.for_cache(case.k, W.SCALE)
    k0, v0 = case.k.clone(), case.v.clone()
    k_new = W.normal_bf16(4501, 40, (2, W.HKV, 6, W.D), DEV)
    v_new = W.normal_bf16(4501, 41, (2, W.HKV, 6, W.D), DEV)
    B.sparrow_kv_append(ctx, k_new, v_new, case.k, case.v, case.kv_len, 6)
    torch.cuda.synchronize()
    for b, n in enumerate(case.kv_len):
        assert torch.equal(case.k[b, :, n:n + 6], k_new[b]) and torch.equal(case.v[b, :, n:n + 6], v_new[b])
        k0[b, :, n:n + 6] = k_new[b]
        v0[b, :, n:n + 6] = v_new[b]
    assert torch.equal(case.k, k0) and torch.equal(case.v, v0)          # nothing else was touched
    with pytest.raises(B.SparrowError):
        B.sparrow_kv_append(ctx, k_new, v_new, case.k, case.v, [396, 10], 6)     # 396 + 6 > capacity


def test_compacted_anchors_are_a_bit_exact_gather_and_serve_the_verify_kernel():
    """Compacting the anchored rows and running the verification kernel on the short cache is the
    anchored mode without a lower window bound: same oracle, contiguous stream instead of a gather."""
    T = 10
    ac = anchor_case(4600, 3000, [[40, 2600]], 0, T, 2, DEV)
    ctx = B.Context.for_cache(ac.k, W.SCALE)
    cap_c = ac.n_anchor + 7
    kc = torch.zeros((2, W.HKV, cap_c, W.D), dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    B.sparrow_compact_anchors(ctx, ac.k, ac.v, ac.anchor_idx, ac.n_anchor, kc, vc, cap_c, 0)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    rows = ac.anchor_idx[0].long()
    assert torch.equal(kc[:, :, :ac.n_anchor], ac.k[:, :, rows]) and torch.equal(vc[:, :, :ac.n_anchor], ac.v[:, :, rows])
    assert not kc[:, :, ac.n_anchor:].any()
    # tree among the draft rows, all text anchors visible: the verification kernel on the compact cache
    parents = torch.tensor([W.random_tree_parents(4601 + b, 99, T) for b in range(2)], dtype=torch.int32, device=DEV)
    cctx = B.Context.for_cache(kc, W.SCALE)
    out = torch.full_like(ac.q, float("nan"))
    lse = torch.full((2, W.HQ, T), float("nan"), dtype=torch.float32, device=DEV)
    B.sparrow_verify_attn(cctx, ac.q, kc, vc, [ac.n_anchor - T] * 2, parents, T, out, lse)
    torch.cuda.synchronize()
    assert cctx.last_device_status() == 0
    ref_out, ref_lse = oracle.anchor_attn_tree(W.bf16_bits(ac.q), W.bf16_bits(ac.k), W.bf16_bits(ac.v),
                                               ac.anchor_idx.cpu().numpy(), 0, parents.cpu().numpy(), W.SCALE)
    check(out, lse, ref_out, ref_lse)


def test_compact_anchors_reports_a_bad_index_and_writes_zeros():
    ac = anchor_case(4700, 600, [[10, 500]], 0, 4, 1, DEV)
    ctx = B.Context.for_cache(ac.k, W.SCALE)
    idx = ac.anchor_idx.clone()
    idx[0, 3] = ac.capacity + 5
    kc = torch.ones((1, W.HKV, ac.n_anchor, W.D), dtype=torch.bfloat16, device=DEV)
    vc = torch.ones_like(kc)
    B.sparrow_compact_anchors(ctx, ac.k, ac.v, idx, ac.n_anchor, kc, vc, ac.n_anchor, 0)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 4                      # SPARROW_ERR_ANCHOR
    assert not kc[:, :, 3].any() and not vc[:, :, 3].any()
    assert torch.equal(kc[:, :, 4], ac.k[:, :, int(idx[0, 4])])
    with pytest.raises(B.SparrowError):
        B.sparrow_compact_anchors(ctx, ac.k, ac.v, idx, ac.n_anchor, kc, vc, ac.n_anchor, 1)     # does not fit
