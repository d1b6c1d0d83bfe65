"""GPU tests of how calls are ordered: back-to-back fused calls (programmatic dependent launch with
counter-ordered writes), the stream-ordered two-kernel mode, calls captured into a CUDA graph, and
the bounded device-side wait.  Results are always compared with the CPU oracle."""
import os

import numpy as np
import pytest
import torch

from paper_2602_15318_b200 import binding as B
from paper_2602_15318_b200 import workloads as W

from gpu_util import anchor_case, check, oracle_verify, run_verify

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _overlapping_ctx(k_cache):
    """A context whose single calls may start early behind its previous call (the tests here
    enqueue nothing in between that could break the rule this opt-in states)."""
    ctx = B.Context.for_cache(k_cache, W.SCALE)
    ctx.set_call_overlap(True)
    return ctx


def _new(case):
    out = torch.full_like(case.q, float("nan"))
    lse = torch.full((case.B, W.HQ, case.T), float("nan"), dtype=torch.float32, device=DEV)
    return out, lse


def test_back_to_back_calls_keep_their_results_apart():
    """Many calls enqueued without any synchronisation, alternating between inputs with different
    shapes of work (several pieces / single piece, one and two row blocks) on one context: every
    call's outputs must be its own."""
    cap = 3000 + 64
    cases = [W.make_verify_case(500 + i, kv, T, tree, DEV, capacity=cap)
             for i, (kv, T, tree) in enumerate([([3000], 16, "chain"), ([90], 5, "random"), ([2500], 24, "random"),
                                                ([1700], 8, "chain"), ([40], 19, "chain")])]
    refs = [oracle_verify(c) for c in cases]
    ctx = _overlapping_ctx(cases[0].k)
    results = []
    for rep in range(6):
        for c in cases:
            out, lse = _new(c)
            B.sparrow_verify_attn(ctx, c.q, c.k, c.v, c.kv_len, c.parents, c.T, out, lse)
            results.append((out, lse))
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    for i, (out, lse) in enumerate(results):
        check(out, lse, *refs[i % len(cases)])


def test_same_output_buffer_reused_by_consecutive_calls():
    """Calls that write the same out / lse buffers land in call order: after the stream drains the
    buffers hold the last call's result."""
    a = W.make_verify_case(601, [2800], 12, "random", DEV)
    b = W.make_verify_case(602, [2800], 12, "chain", DEV)
    ctx = _overlapping_ctx(a.k)
    out, lse = _new(a)
    for _ in range(5):
        B.sparrow_verify_attn(ctx, a.q, a.k, a.v, a.kv_len, a.parents, a.T, out, lse)
        B.sparrow_verify_attn(ctx, b.q, b.k, b.v, b.kv_len, b.parents, b.T, out, lse)
    torch.cuda.synchronize()
    check(out, lse, *oracle_verify(b))
    B.sparrow_verify_attn(ctx, a.q, a.k, a.v, a.kv_len, a.parents, a.T, out, lse)
    torch.cuda.synchronize()
    check(out, lse, *oracle_verify(a))


def test_anchor_and_verify_calls_interleave():
    v = W.make_verify_case(603, [2000], 8, "chain", DEV, capacity=2100)
    a = anchor_case(604, 2000, [[50, 1800]], 0, 8, 1, DEV, capacity=2100)
    ctx = _overlapping_ctx(v.k)
    outs = []
    for _ in range(3):
        ov, lv = _new(v)
        B.sparrow_verify_attn(ctx, v.q, v.k, v.v, v.kv_len, v.parents, v.T, ov, lv)
        oa, la = _new(a)
        B.sparrow_anchor_attn(ctx, a.q, a.k, a.v, a.anchor_idx, a.n_anchor, a.window, a.T, oa, la)
        outs.append((ov, lv, oa, la))
    torch.cuda.synchronize()
    import oracle
    ra = oracle.anchor_attn(W.bf16_bits(a.q), W.bf16_bits(a.k), W.bf16_bits(a.v), a.anchor_idx.cpu().numpy(), a.window, W.SCALE)
    rv = oracle_verify(v)
    for ov, lv, oa, la in outs:
        check(ov, lv, *rv)
        check(oa, la, *ra)


def test_stream_ordered_mode(monkeypatch):
    """SPARROW_NO_PDL=1 at context creation: every call is ordered by the stream alone and touches no
    counter -- the split-KV pass and, where a sequence has several pieces, the combine kernel."""
    monkeypatch.setenv("SPARROW_NO_PDL", "1")
    for kv, T, tree in [([3000, 1500], 12, "random"), ([129], 19, "random"), ([64], 8, "chain")]:
        case = W.make_verify_case(610 + T, kv, T, tree, DEV)
        ctx = _overlapping_ctx(case.k)
        n0 = ctx.launch_count()
        out, lse, _ = run_verify(case, ctx)
        assert ctx.launch_count() - n0 == (2 if max(kv) + T > 128 else 1)
        check(out, lse, *oracle_verify(case))


def test_call_captured_into_a_graph_replays():
    case = W.make_verify_case(620, [2500, 900], 10, "random", DEV)
    ctx = _overlapping_ctx(case.k)
    out, lse = _new(case)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        B.sparrow_verify_attn(ctx, case.q, case.k, case.v, case.kv_len, case.parents, case.T, out, lse)   # warm-up
    s.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        B.sparrow_verify_attn(ctx, case.q, case.k, case.v, case.kv_len, case.parents, case.T, out, lse, stream=s)
    ref = oracle_verify(case)
    for _ in range(3):
        out.fill_(float("nan")); lse.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        check(out, lse, *ref)
    # ordinary calls after the replays still work on the same context
    out2, lse2, _ = run_verify(case, ctx)
    check(out2, lse2, *ref)


def test_bounded_wait_gives_up_and_context_survives():
    case = W.make_verify_case(630, [1500], 8, "chain", DEV)
    ctx = _overlapping_ctx(case.k)
    out, lse, _ = run_verify(case, ctx)
    B.sparrow_debug_wait_counter(ctx, 0)                  # everything it waits for has happened
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    B.sparrow_debug_wait_counter(ctx, 5)                  # nothing will ever bump the counter that far
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 7                  # SPARROW_ERR_TIMEOUT, then cleared
    assert ctx.status_word() == 4 | (1 << 16)             # timeout bit + the debug wait's site bit
    assert ctx.last_device_status() == 0
    out2, lse2, _ = run_verify(case, ctx)
    check(out2, lse2, *oracle_verify(case))


def test_plan_policy_changes_between_calls():
    """The policy only changes how the key range is cut: every policy meets the tolerances, the
    policy may change between two calls of a stream without any synchronisation, and a long
    stream of calls with few, long pieces (many calls resident at once) keeps every result apart."""
    cap = 9000 + 64
    cases = [W.make_verify_case(700 + i, kv, T, tree, DEV, capacity=cap)
             for i, (kv, T, tree) in enumerate([([9000], 16, "chain"), ([5000], 30, "random"), ([7000], 8, "chain")])]
    refs = [oracle_verify(c) for c in cases]
    ctx = _overlapping_ctx(cases[0].k)
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    targets = {}
    for pol in (B.PLAN_LATENCY, B.PLAN_BALANCED, B.PLAN_THROUGHPUT):
        ctx.set_plan_policy(pol)
        targets[pol] = ctx.plan_target_items()
    assert targets[B.PLAN_LATENCY] == n_sm
    assert targets[B.PLAN_LATENCY] > targets[B.PLAN_BALANCED] > targets[B.PLAN_THROUGHPUT] >= 1
    with pytest.raises(B.SparrowError):
        ctx.set_plan_policy(17)
    results = []
    for rep in range(40):
        ctx.set_plan_policy((B.PLAN_THROUGHPUT, B.PLAN_LATENCY, B.PLAN_THROUGHPUT, B.PLAN_BALANCED)[rep % 4])
        for c in cases:
            out, lse = _new(c)
            B.sparrow_verify_attn(ctx, c.q, c.k, c.v, c.kv_len, c.parents, c.T, out, lse)
            results.append((out, lse))
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    for i, (out, lse) in enumerate(results):
        check(out, lse, *refs[i % len(cases)])


@pytest.mark.parametrize("policy", [B.PLAN_LATENCY, B.PLAN_BALANCED, B.PLAN_THROUGHPUT])
def test_long_stream_is_bitwise_reproducible(policy):
    """Thousands of calls queued back to back over rotating caches, several calls resident at
    once: every call must reproduce, bit for bit, what the same call gave when it ran alone (any
    ordering mistake between overlapping calls shows up as a changed bit or a timeout)."""
    cap = 20000 + 32
    cases = [W.make_verify_case(800 + i, [20000 - 37 * i], 16, "chain", DEV, capacity=cap) for i in range(3)]
    ctx = _overlapping_ctx(cases[0].k)
    ctx.set_plan_policy(policy)
    alone = []
    for c in cases:                                # (each call alone on the GPU: the stream is drained after it)
        out, lse = _new(c)
        B.sparrow_verify_attn(ctx, c.q, c.k, c.v, c.kv_len, c.parents, c.T, out, lse)
        torch.cuda.synchronize()
        alone.append((out, lse))
    check(alone[0][0], alone[0][1], *oracle_verify(cases[0]))
    n_slots = 12                                   # output buffers in rotation: more than the calls in flight
    outs = [[_new(c) for _ in range(n_slots)] for c in cases]
    batch = B.VerifyBatch([(c.q, c.k, c.v, c.kv_len, c.parents, c.T, outs[i][s][0], outs[i][s][1])
                           for s in range(n_slots) for i, c in enumerate(cases)])
    for rep in range(60):                          # 60 x 36 calls
        B.sparrow_verify_attn_batch(ctx, batch)
        if rep % 20 == 19:
            torch.cuda.synchronize()
            for i in range(len(cases)):
                for s in range(n_slots):
                    assert torch.equal(outs[i][s][0], alone[i][0]) and torch.equal(outs[i][s][1], alone[i][1])
                    outs[i][s][0].zero_()
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0


def test_whole_step_in_one_stream_without_synchronisation():
    """Append draft rows, verify, accept, keep the accepted rows, append the next draft block and
    verify again -- everything enqueued on one stream with no host synchronisation in between.
    The second verification must see the cache exactly as the row moves left it (fused calls
    overlap their neighbours; the plain kernels in between must still be ordered)."""
    import oracle
    T, kv0 = 12, 3000
    case = W.make_verify_case(900, [kv0], T, "random", DEV, capacity=kv0 + 3 * T)
    ctx = _overlapping_ctx(case.k)
    ctx.set_plan_policy(B.PLAN_THROUGHPUT)
    d = lambda x: torch.tensor(x, dtype=torch.int32, device=DEV)
    par = case.parents[0].tolist()
    # synthetic tokens: the chain 0 -> first child -> ... is "right", everything else wrong
    nxt = [100 + i for i in range(T + 1)]
    tok = [nxt[par[i] + 1] if (par[i] == -1 or i == min(c for c in range(T) if par[c] == par[i])) else -5 for i in range(T)]
    ref_path, _ = oracle.greedy_accept(tok, par, nxt)
    assert len(ref_path) >= 2
    k_new = W.normal_bf16(901, 40, (1, W.HKV, T, W.D), DEV)
    v_new = W.normal_bf16(901, 41, (1, W.HKV, T, W.D), DEV)
    k_new2 = W.normal_bf16(902, 40, (1, W.HKV, T, W.D), DEV)
    v_new2 = W.normal_bf16(902, 41, (1, W.HKV, T, W.D), DEV)
    q2 = W.normal_bf16(903, 42, (1, T, W.HQ, W.D), DEV)
    out1, lse1 = _new(case)
    out2, lse2 = _new(case)
    path = torch.empty((1, T), dtype=torch.int32, device=DEV)
    n_acc = torch.empty((1,), dtype=torch.int32, device=DEV)
    bonus = torch.empty((1,), dtype=torch.int32, device=DEV)
    kv1 = kv0 + len(ref_path)                    # (known here because the tokens are synthetic)
    B.sparrow_kv_append(ctx, k_new, v_new, case.k, case.v, [kv0], T)
    B.sparrow_verify_attn(ctx, case.q, case.k, case.v, [kv0], case.parents, T, out1, lse1)
    B.sparrow_accept_greedy(ctx, d([tok]), case.parents, d([nxt]), T, path, n_acc, bonus)
    B.sparrow_kv_keep_accepted(ctx, case.k, case.v, [kv0], path, n_acc, T)
    B.sparrow_kv_append(ctx, k_new2, v_new2, case.k, case.v, [kv1], T)
    B.sparrow_verify_attn(ctx, q2, case.k, case.v, [kv1], case.parents, T, out2, lse2)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    assert int(n_acc[0]) == len(ref_path) and path[0, :len(ref_path)].tolist() == ref_path
    # the same sequence of cache states on the host
    host = W.make_verify_case(900, [kv0], T, "random", "cpu", capacity=kv0 + 3 * T)
    k_ref, v_ref = host.k.clone(), host.v.clone()
    k_ref[0, :, kv0:kv0 + T] = k_new[0].cpu(); v_ref[0, :, kv0:kv0 + T] = v_new[0].cpu()
    r1 = oracle.verify_attn(W.bf16_bits(case.q), W.bf16_bits(k_ref), W.bf16_bits(v_ref), [kv0], [par], W.SCALE)
    check(out1, lse1, *r1)
    k_old, v_old = k_ref.clone(), v_ref.clone()
    for i, node in enumerate(ref_path):
        k_ref[0, :, kv0 + i] = k_old[0, :, kv0 + node]; v_ref[0, :, kv0 + i] = v_old[0, :, kv0 + node]
    k_ref[0, :, kv1:kv1 + T] = k_new2[0].cpu(); v_ref[0, :, kv1:kv1 + T] = v_new2[0].cpu()
    assert torch.equal(case.k[0, :, :kv1 + T].cpu(), k_ref[0, :, :kv1 + T])
    r2 = oracle.verify_attn(W.bf16_bits(q2), W.bf16_bits(k_ref), W.bf16_bits(v_ref), [kv1], [par], W.SCALE)
    check(out2, lse2, *r2)


def test_calls_of_two_contexts_on_one_stream_take_stream_order():
    """A call that follows a call of ANOTHER context must not start early (the other context's
    writes are invisible to this context's counters): here its queries are the other call's output."""
    T = 16
    a = W.make_verify_case(950, [9000], T, "chain", DEV)
    b = W.make_verify_case(951, [7000], T, "random", DEV)
    ctx_a = _overlapping_ctx(a.k)
    ctx_b = _overlapping_ctx(b.k)
    out_a, lse_a = _new(a)
    out_b, lse_b = _new(b)
    for _ in range(5):
        out_a.fill_(float("nan"))
        B.sparrow_verify_attn(ctx_a, a.q, a.k, a.v, a.kv_len, a.parents, T, out_a, lse_a)
        B.sparrow_verify_attn(ctx_b, out_a, b.k, b.v, b.kv_len, b.parents, T, out_b, lse_b)     # q = the other call's out
        torch.cuda.synchronize()
        again, lse_again = _new(b)
        B.sparrow_verify_attn(ctx_b, out_a, b.k, b.v, b.kv_len, b.parents, T, again, lse_again)
        torch.cuda.synchronize()
        assert torch.isfinite(out_b.float()).all()
        assert torch.equal(out_b, again) and torch.equal(lse_b, lse_again)
    assert ctx_a.last_device_status() == 0 and ctx_b.last_device_status() == 0


# ---- what may start early, and what may not ---------------------------------------------------

def test_call_behind_a_foreign_kernel_with_an_early_trigger_waits_for_it():
    """A kernel that is not the library's sits between two calls; it lets its dependents launch at
    once and writes the next call's q only much later.  The call must still see that q."""
    T = 16
    a = W.make_verify_case(960, [6000], T, "chain", DEV)
    b = W.make_verify_case(961, [6000], T, "random", DEV, capacity=a.capacity)
    ref_b = oracle_verify(b)
    ctx = B.Context.for_cache(a.k, W.SCALE)           # default: single calls take plain stream order
    q_live = torch.zeros_like(b.q)
    out_a, lse_a = _new(a)
    for delay in (0, 50, 400):
        q_live.zero_()
        out_b, lse_b = _new(b)
        B.sparrow_verify_attn(ctx, a.q, a.k, a.v, a.kv_len, a.parents, T, out_a, lse_a)
        B.sparrow_debug_early_trigger_copy(ctx, b.q, q_live, b.q.numel() * 2, delay)
        B.sparrow_verify_attn(ctx, q_live, b.k, b.v, b.kv_len, b.parents, T, out_b, lse_b)
        torch.cuda.synchronize()
        check(out_b, lse_b, *ref_b)
    assert ctx.last_device_status() == 0


@pytest.mark.parametrize("gap", [1, 2, 5])
@pytest.mark.parametrize("policy", [B.PLAN_LATENCY, B.PLAN_THROUGHPUT])
def test_call_reading_an_earlier_calls_output_is_not_started_early(gap, policy):
    """Inside one batch (calls start early behind each other) call n reads, as its q, the out of
    call n - gap, with other calls in between: the library must notice and order that launch.
    The result must equal, bit for bit, what the same chain gives with a synchronisation after
    every call."""
    T, n_calls = 16, 12
    cases = [W.make_verify_case(970 + i, [9000 - 100 * i], T, "chain", DEV, capacity=9100) for i in range(3)]
    ctx = B.Context.for_cache(cases[0].k, W.SCALE)
    ctx.set_plan_policy(policy)

    def run(sync_every_call):
        outs = [_new(cases[0]) for _ in range(n_calls)]
        calls = []
        for n in range(n_calls):
            c = cases[n % 3]
            q = c.q if n < gap else outs[n - gap][0]
            calls.append((q, c.k, c.v, c.kv_len, c.parents, T, outs[n][0], outs[n][1]))
        if sync_every_call:
            for call in calls:
                B.sparrow_verify_attn_batch(ctx, B.VerifyBatch([call]))
                torch.cuda.synchronize()
        else:
            B.sparrow_verify_attn_batch(ctx, B.VerifyBatch(calls))
            torch.cuda.synchronize()
        return outs

    want = run(True)
    for _ in range(3):
        got = run(False)
        for (o, l), (wo, wl) in zip(got, want):
            assert torch.equal(o, wo) and torch.equal(l, wl)
    assert ctx.last_device_status() == 0


def test_many_caches_through_one_context():
    """More distinct K / V / q buffers than the context's tensor-map cache holds, revisited in an
    order that mixes hits with evictions: every call must use the maps of its own buffers."""
    T, kv, n_buf = 4, 200, 1400
    base = W.make_verify_case(980, [kv], T, "chain", DEV, capacity=256)
    ks = W.normal_bf16(981, 2, (n_buf, W.HKV, 256, W.D), DEV)
    vs = W.normal_bf16(981, 3, (n_buf, W.HKV, 256, W.D), DEV)
    qs = W.normal_bf16(981, 1, (n_buf, T, W.HQ, W.D), DEV)
    ctx = B.Context.for_cache(base.k, W.SCALE)
    outs = torch.full((n_buf, T, W.HQ, W.D), float("nan"), dtype=torch.bfloat16, device=DEV)
    lses = torch.full((n_buf, W.HQ, T), float("nan"), dtype=torch.float32, device=DEV)
    order = list(range(n_buf)) + [0, 777, 1, 1399, 2, 640] + list(range(0, n_buf, 7))
    for i in order:
        B.sparrow_verify_attn(ctx, qs[i:i + 1], ks[i:i + 1], vs[i:i + 1], [kv], base.parents, T, outs[i:i + 1], lses[i:i + 1])
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    import oracle
    for i in (0, 1, 2, 640, 777, 1398, 1399):
        ref = oracle.verify_attn(W.bf16_bits(qs[i:i + 1]), W.bf16_bits(ks[i:i + 1]), W.bf16_bits(vs[i:i + 1]), [kv],
                                 base.parents.cpu().numpy(), W.SCALE)
        check(outs[i:i + 1], lses[i:i + 1], *ref)
    first = outs.clone()
    for i in reversed(order):
        B.sparrow_verify_attn(ctx, qs[i:i + 1], ks[i:i + 1], vs[i:i + 1], [kv], base.parents, T, outs[i:i + 1], lses[i:i + 1])
    torch.cuda.synchronize()
    assert torch.equal(first, outs)


def test_plan_log_line(monkeypatch, capfd):
    """SPARROW_LOG=1 at context creation: one line per verification call on stderr."""
    monkeypatch.setenv("SPARROW_LOG", "1")
    case = W.make_verify_case(990, [3000], 20, "random", DEV)
    out, lse, ctx = run_verify(case)
    check(out, lse, *oracle_verify(case))
    err = capfd.readouterr().err
    assert "[sparrow] verify call" in err and "2 row block(s)" in err and "keys [0, 3020)" in err


def test_timeline_tool_runs_and_sees_every_cta():
    """The stamped build runs the same kernels: a short C1 timeline reports one row per phase and
    the CTA count of the latency policy's plan."""
    import subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "paper_2602_15318_b200.timeline", "--config", "C1", "--calls", "8"],
                       cwd=root, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = r.stdout.strip().splitlines()
    assert "CTAs" in lines[0] and int(lines[0].split(":")[1].split("CTAs")[0]) > 1
    for phase in ("kernel entered", "partial rows stored", "finisher: merged rows written", "leaving"):
        assert any(l.startswith(phase) for l in lines), phase
