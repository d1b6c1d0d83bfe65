"""Helpers shared by the GPU parity tests: run a case through the C ABI, run the oracle on the
same tensors, compare within the stated tolerances."""
import numpy as np
import torch

import oracle
from paper_2602_15318_b200 import binding as B
from paper_2602_15318_b200 import workloads as W

TOL_OUT = 1e-2      # max |out_gpu - out_oracle|   (bf16 inputs, fp32 accumulation, bf16 output)
TOL_LSE = 1e-3      # max |lse_gpu - lse_oracle|


def run_verify(case: W.VerifyCase, ctx=None, policy=None):
    ctx = ctx or B.Context.for_cache(case.k, W.SCALE, n_q_heads=case.q.shape[2])
    if policy is not None:
        ctx.set_plan_policy(policy)
    out = torch.full_like(case.q, float("nan"))
    lse = torch.full((case.B, case.q.shape[2], case.T), float("nan"), dtype=torch.float32, device=case.q.device)
    B.sparrow_verify_attn(ctx, case.q, case.k, case.v, case.kv_len, case.parents, case.T, out, lse)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    return out, lse, ctx


def run_anchor(case: W.AnchorCase, ctx=None):
    ctx = ctx or B.Context.for_cache(case.k, W.SCALE)
    out = torch.full_like(case.q, float("nan"))
    lse = torch.full((case.B, W.HQ, case.T), float("nan"), dtype=torch.float32, device=case.q.device)
    B.sparrow_anchor_attn(ctx, case.q, case.k, case.v, case.anchor_idx, case.n_anchor, case.window,
                          case.T, out, lse)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    return out, lse, ctx


def anchor_case(seed, seq_len, vis_spans, window, T, batch=1, device="cuda:0", capacity=None, name=""):
    """An anchored-mode case whose anchor list is the oracle's (Eq. 2's index set under the window
    reading): text positions of [0, seq_len) within the last `window` positions, then the T draft rows."""
    idx = oracle.anchor_idx(seq_len, vis_spans, window, T).tolist()
    return W.make_anchor_case(seed, idx, window, T, batch, device,
                              capacity=capacity if capacity is not None else seq_len + T, name=name)


def oracle_verify(case: W.VerifyCase, rows=None):
    return oracle.verify_attn(W.bf16_bits(case.q), W.bf16_bits(case.k), W.bf16_bits(case.v),
                              case.kv_len, case.parents.cpu().numpy(), W.SCALE, rows=rows)


def oracle_anchor(case: W.AnchorCase, rows=None):
    return oracle.anchor_attn(W.bf16_bits(case.q), W.bf16_bits(case.k), W.bf16_bits(case.v),
                              case.anchor_idx.cpu().numpy(), case.window, W.SCALE, rows=rows)


def compare(out, lse, ref_out, ref_lse, rows=None):
    """Element-by-element comparison; returns (max |d out|, max |d lse|)."""
    o = out.double().cpu().numpy()
    l = lse.double().cpu().numpy()
    if rows is not None:
        o = np.stack([o[b, t, h] for b, t, h in rows])
        l = np.array([l[b, h, t] for b, t, h in rows])
    assert not np.isnan(o).any() and not np.isnan(l).any()
    both_inf = np.isinf(l) & np.isinf(ref_lse) & (l == ref_lse)
    d_out = float(np.max(np.abs(o - ref_out)))
    d_lse = float(np.max(np.where(both_inf, 0.0, np.abs(l - ref_lse)))) if l.size else 0.0
    return d_out, d_lse


def check(out, lse, ref_out, ref_lse, rows=None):
    d_out, d_lse = compare(out, lse, ref_out, ref_lse, rows)
    print(f"[parity] max|d out| = {d_out:.3e}  max|d lse| = {d_lse:.3e}  ({ref_lse.size} rows)")     # shown by pytest -s
    assert d_out <= TOL_OUT, f"max |d out| = {d_out}"
    assert d_lse <= TOL_LSE, f"max |d lse| = {d_lse}"
    return d_out, d_lse


def sample_rows(seed, B_, T, n):
    """Seeded sample of (b, t, h) triples, always including the corners."""
    g = W.host_stream(seed, 9)
    rows = {(0, 0, 0), (B_ - 1, T - 1, W.HQ - 1), (0, T - 1, 0), (B_ - 1, 0, W.HQ - 1)}
    while len(rows) < n:
        rows.add((next(g) % B_, next(g) % T, next(g) % W.HQ))
    return sorted(rows)
