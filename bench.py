#!/usr/bin/env python
"""Benchmark of the speculative-step attention path.

Headline (the metric quoted on the long-video configuration): verification attention, batch 1,
28/4 heads, head_dim 128, KV length 26,112 (25,600 visual + 512 text), T = 16 chain, bf16.
A step = one sparrow_verify_attn call (split-KV pass + LSE combine).  Steps rotate over R distinct
K/V caches whose total size is several times the L2 capacity, so every step streams its cache
from HBM.  Timing is by CUDA events on the launching stream, after warm-up, synchronised on both
sides; the calls are enqueued from C (sparrow_verify_attn_batch) so Python is not in the loop.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--all-configs]

Prints ONE JSON line on stdout.  With --gpus N > 1 (launched under torch.distributed.run) every
rank runs an independent replica on its own GPU -- the path has no cross-GPU exchange -- and the
reported time is the maximum over ranks.
"""
import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verify_attn_us_per_call_kv26112_T16_bf16"
UNIT = "us"
WORKLOAD = "C2: verify attention, batch 1, 28/4 heads, head_dim 128, kv_len 26112, T=16 chain"
L2_BYTES_FALLBACK = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json)", d
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)", {}


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons of one GPU while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"], "samples": 0}
        # keep the samples taken under load (upper half of the observed clocks)
        sm_sorted = sorted(sm)
        return {"sm_mhz": sm_sorted[len(sm_sorted) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def kernel_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for f in ("verify_tc.cuh", "common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2602_15318_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def profiled_traffic():
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, or None when
    the kernel sources have changed since that capture."""
    p = os.path.join(ROOT, "profiles", "verify_tc_kernel_c2.md")
    try:
        text = open(p).read()
        import re
        t = re.search(r"traffic_bytes_per_launch:\s*(\d+)", text)
        h = re.search(r"kernel_sources_sha256:\s*([0-9a-f]{64})", text)
        if t and h and h.group(1) == kernel_sources_sha256():
            return int(t.group(1))
    except Exception:
        pass
    return None


def max_over_ranks(value, dist, device="cpu"):
    """Maximum of a per-rank scalar over the process group (identity without one)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def oracle_time_c2(min_seconds=8.0, max_reps=40):
    """Times the CPU oracle, as it stands, on full C2 calls (all 448 (token, head) rows)."""
    import oracle
    from paper_2602_15318_b200 import workloads as W
    case = W.make_config(1, "cpu")
    qb, kb, vb = W.bf16_bits(case.q), W.bf16_bits(case.k), W.bf16_bits(case.v)
    par = case.parents.numpy()
    cores = oracle.host_threads()
    oracle.verify_attn(qb, kb, vb, case.kv_len, par, W.SCALE, rows=[(0, 0, 0)])      # loads the library
    reps, t0 = 0, time.perf_counter()
    while True:
        oracle.verify_attn(qb, kb, vb, case.kv_len, par, W.SCALE, n_threads=cores)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or reps >= max_reps:
            break
    return dt / reps * 1e6, cores, reps


def run_reference(args, rank):
    """The reference arm of this build is the CPU oracle timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    import oracle
    from paper_2602_15318_b200 import workloads as W
    case = W.make_config(1, "cpu")
    qb, kb, vb = W.bf16_bits(case.q), W.bf16_bits(case.k), W.bf16_bits(case.v)
    par = case.parents.numpy()
    cores = oracle.host_threads()
    # a step = a bounded sample of one C2 call: 56 of its 448 (token, head) rows, scaled up
    rows = [(0, t, h) for t in range(0, 16, 2) for h in range(0, 28, 4)]
    scale_up = 448.0 / len(rows)
    for _ in range(min(warmup, 3)):
        oracle.verify_attn(qb, kb, vb, case.kv_len, par, W.SCALE, rows=rows, n_threads=cores)
    steps = min(steps, 200)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.verify_attn(qb, kb, vb, case.kv_len, par, W.SCALE, rows=rows, n_threads=cores)
    dt = time.perf_counter() - t0
    us = dt / steps * scale_up * 1e6
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(warmup, 3), "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD},
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{len(rows)} of 448 (token, head) rows per step, scaled by {scale_up:g}"},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def time_calls(ctx, batch, n_steps, B, torch):
    """Enqueues n_steps calls (cycling through the prepared batch) between two CUDA events."""
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    R = batch.n
    torch.cuda.synchronize()
    start.record()
    done = 0
    while done < n_steps:
        n = min(R, n_steps - done)
        B.sparrow_verify_attn_batch(ctx, batch, n)
        done += n
    stop.record()
    torch.cuda.synchronize()
    return start.elapsed_time(stop) * 1e3 / n_steps          # us per call


def time_isolated_calls(ctx, cases, outs, lses, n_calls, B, torch, queued=True):
    """Time of one call that overlaps nothing: every call is bracketed by its own pair of events
    and the stream is drained before the next one.  queued=True (what a decoder sees: the host
    runs ahead of the GPU) first enqueues a short spin kernel, so that the two events and the call
    are already in the stream when the GPU reaches them -- the figure is the call's device time
    including its launch gap, without the host's enqueue latency; queued=False starts from an idle
    stream, so the GPU also waits for the host to get the launch through.  Median in us."""
    singles = [B.VerifyBatch([(c.q, c.k, c.v, c.kv_len, c.parents, c.T, o, l)]) for c, o, l in zip(cases, outs, lses)]
    times = []
    for i in range(n_calls):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if queued:
            torch.cuda._sleep(150000)
        e0.record()
        B.sparrow_verify_attn_batch(ctx, singles[i % len(singles)])
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    times.sort()
    return times[len(times) // 2]


def build_rotation(W, B, torch, dev, cfg_index, n_caches, calls_per_batch=1000):
    """R distinct (q, K, V) sets of one configuration, one context sized for them, and one prepared
    array of calls that cycles through them (a whole number of cycles, about calls_per_batch calls):
    inside one sparrow_verify_attn_batch() every call after the first starts early behind its
    predecessor, so a long array keeps the stream of calls overlapped."""
    cases = [W.make_config(cfg_index, dev, layer=r) for r in range(n_caches)]
    ctx = B.Context.for_cache(cases[0].k, W.SCALE)
    outs = [torch.empty_like(c.q) for c in cases]
    lses = [torch.empty((c.B, W.HQ, c.T), dtype=torch.float32, device=dev) for c in cases]
    cycles = max(1, calls_per_batch // n_caches)
    batch = B.VerifyBatch([(c.q, c.k, c.v, c.kv_len, c.parents, c.T, o, l)
                           for c, o, l in zip(cases, outs, lses)] * cycles)
    return cases, ctx, outs, lses, batch


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100000)
    ap.add_argument("--warmup", type=int, default=2000)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--all-configs", action="store_true",
                    help="also time the anchored-mode variants (C4 from a graph, compacted, with a draft tree)")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the other configurations (C1, C3, C4, C5), which are otherwise timed and "
                         "reported under other_configs in the same JSON line")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", choices=["C1", "C2", "C3", "C5", "HSR"],
                    help="time just this configuration's stream of calls (a small run for a profiler capture): "
                         "--steps calls after --warmup calls under --policy, one JSON line")
    ap.add_argument("--policy", choices=["latency", "balanced", "throughput"], default="throughput")
    ap.add_argument("--single-calls", action="store_true",
                    help="with --only: enqueue every call on its own (plain stream order, nothing overlaps)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    from paper_2602_15318_b200 import binding as B
    from paper_2602_15318_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    B.lib()                                   # fails loudly if the CUDA library is not built
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size or L2_BYTES_FALLBACK
    if args.only:
        run_only(args, W, B, torch, dev, l2, steps, warmup)
        return
    probe = W.make_config(1, "cpu")
    kv_bytes, io_bytes, flops = probe.kv_bytes(), probe.io_bytes(), probe.flops()
    n_caches = max(4, -(-4 * l2 // kv_bytes))                 # R * bytes >= 4 x L2
    cases, ctx, outs, lses, batch = build_rotation(W, B, torch, dev, 1, n_caches)
    launches0 = ctx.launch_count()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # -- device-resident throughput: whole calls ------------------------------------------------
    # The timed stream is thousands of independent calls queued back to back, which is what the
    # planner's throughput policy is for; the other policies are timed below and reported beside it.
    ctx.set_plan_policy(B.PLAN_THROUGHPUT)
    time_calls(ctx, batch, warmup, B, torch)
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    t_sample = time.perf_counter()
    launches_before = ctx.launch_count()
    us_call = time_calls(ctx, batch, steps, B, torch)
    launches_timed = ctx.launch_count() - launches_before
    barrier()
    # nvidia-smi needs a second or so to deliver samples: a short timed region is followed by an
    # untimed continuation of the same launches, so that the clocks are still read under this load
    continued = 0
    while time.perf_counter() - t_sample < 1.5:
        time_calls(ctx, batch, 2000, B, torch)
        continued += 2000
    clocks = sampler.stop()
    if continued:
        clocks["note"] = f"timed region shorter than the sampling period: {continued} more untimed calls of the same workload kept the load up while sampling"
    us_call = max_over_ranks(us_call, dist, dev)

    # -- every policy: sustained stream and isolated call (cold cache: the rotation continues) ---
    policies = {}
    for name, pol in POLICIES(B):
        ctx.set_plan_policy(pol)
        if pol == B.PLAN_THROUGHPUT:
            us_stream = us_call
        else:
            time_calls(ctx, batch, 200, B, torch)
            us_stream = max_over_ranks(time_calls(ctx, batch, max(2000, steps // 4), B, torch), dist, dev)
        policies[name] = {"target_items": ctx.plan_target_items(), "us_per_call_stream": us_stream,
                          "us_per_call_isolated": time_isolated_calls(ctx, cases, outs, lses, 300, B, torch),
                          "us_per_call_isolated_idle_stream": time_isolated_calls(ctx, cases, outs, lses, 100, B, torch, queued=False)}
    us_isolated = policies["latency"]["us_per_call_isolated"]
    ctx.set_plan_policy(B.PLAN_THROUGHPUT)

    # -- L2-warm figure (one cache, labelled as such) --------------------------------------------
    warm = B.VerifyBatch([(cases[0].q, cases[0].k, cases[0].v, cases[0].kv_len, cases[0].parents,
                           cases[0].T, outs[0], lses[0])] * 500)
    time_calls(ctx, warm, 500, B, torch)
    us_warm = time_calls(ctx, warm, max(2000, steps // 10), B, torch)

    # -- the same rotation replayed from a CUDA graph (captured calls run in stream-ordered mode:
    #    split-KV kernel, then combine kernel, one wave of pieces) -------------------------------
    us_graph = None
    try:
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            B.sparrow_verify_attn_batch(ctx, batch, len(cases), stream=side)
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                B.sparrow_verify_attn_batch(ctx, batch, len(cases), stream=side)
            graph.replay(); side.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_rep = 40
            g0.record(side)
            for _ in range(n_rep):
                graph.replay()
            g1.record(side); side.synchronize()
        us_graph = g0.elapsed_time(g1) * 1e3 / (n_rep * len(cases))
        del graph
    except Exception as e:                                   # reported, never fatal for the headline
        us_graph = f"unavailable: {type(e).__name__}"

    # -- end to end through the host-buffer entry point -----------------------------------------
    c0 = cases[0]
    T = c0.T
    q_h = c0.q.cpu().pin_memory()
    k_new = torch.stack([c0.k[b, :, n:n + T, :] for b, n in enumerate(c0.kv_len)]).cpu().pin_memory()
    v_new = torch.stack([c0.v[b, :, n:n + T, :] for b, n in enumerate(c0.kv_len)]).cpu().pin_memory()
    par_h = c0.parents.cpu().pin_memory()
    out_h = torch.empty_like(q_h).pin_memory()
    lse_h = torch.empty((c0.B, W.HQ, T), dtype=torch.float32).pin_memory()
    h2d = q_h.numel() * 2 + k_new.numel() * 2 + v_new.numel() * 2 + par_h.numel() * 4
    d2h = out_h.numel() * 2 + lse_h.numel() * 4
    e2e_steps = max(300, min(steps // 20, 5000))

    ctx.set_plan_policy(B.PLAN_LATENCY)          # every step is synchronised: nothing to overlap with

    def e2e_loop(n):
        for i in range(n):
            c = cases[i % len(cases)]
            B.sparrow_verify_step_host(ctx, q_h, k_new, v_new, c.k, c.v, c.kv_len, par_h, T, out_h, lse_h)
    e2e_loop(20)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    t0 = time.perf_counter()
    e2e_loop(e2e_steps)
    ev1.record()
    torch.cuda.synchronize()
    us_e2e = max(ev0.elapsed_time(ev1) * 1e3, (time.perf_counter() - t0) * 1e6) / e2e_steps
    us_e2e = max_over_ranks(us_e2e, dist, dev)
    status = ctx.last_device_status()
    if status != 0:
        raise SystemExit(f"device status {status} (word {ctx.status_word():#x}) after the timed region")

    peak, peak_kind, peaks = measured_peaks()
    # overhead outside the algorithmic bytes: partial rows (272 B) written once and read once through L2
    tgt = policies["throughput"]["target_items"]
    splits, n_items = B.sparrow_plan_splits(tgt, W.HKV, [n + cases[0].T for n in cases[0].kv_len], cases[0].T)
    partial_bytes = 2 * n_items * 7 * cases[0].T * 272
    alg_bytes = kv_bytes + io_bytes
    achieved = alg_bytes / (us_call * 1e-6) / 1e9
    traffic = profiled_traffic()

    line = {
        "metric": METRIC, "value": us_call, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": us_call / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2_policy": f"rotation over {n_caches} distinct K/V caches "
                   f"({n_caches * kv_bytes / 1e6:.0f} MB > 4 x L2 {l2 / 1e6:.0f} MB)",
                   "launch": "plain stream launches enqueued from C (sparrow_verify_attn_batch)",
                   "plan_policy": "throughput (sparrow_set_plan_policy; the default is balanced)",
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "hbm_gbs_per_call": alg_bytes / (us_call * 1e-6) / 1e9,
        "pct_of_8tbs_nominal": 100.0 * alg_bytes / (us_call * 1e-6) / 8e12,
        "tflops_per_call": flops / (us_call * 1e-6) / 1e12,
        "pct_of_bf16_burst_peak": (100.0 * flops / (us_call * 1e-6) / 1e12 / peaks["bf16_tflops"]) if peaks.get("bf16_tflops") else None,
        "pct_of_bf16_sustained_peak": (100.0 * flops / (us_call * 1e-6) / 1e12 / peaks["bf16_tflops_sustained"])
        if peaks.get("bf16_tflops_sustained") else None,
        "us_per_call_graph_replay": us_graph,
        "partials_bytes_per_call": partial_bytes,
        "us_per_call_isolated": us_isolated,
        "us_per_call_isolated_what": "one call under the latency policy that overlaps no other call: events around the call, "
                                     "enqueued behind a short spin kernel so the host's launch latency is not in the figure "
                                     "(us_per_call_isolated_idle_stream in policies: the same from an idle stream, host latency included); median",
        "policies": policies,
        "us_per_call_l2_warm": us_warm,
        "calls_per_s_all_gpus": world * 1e6 / us_call,
        "roofline": {"bound": "hbm", "kernel": "verify_tc_kernel<1> (the only kernel of a step: split-KV pass with the combine "
                     "fused in); duration = timed region / its launches, back-to-back launches overlapped by "
                     "programmatic dependent launch",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_source": "of " + peak_kind, "algorithmic_bytes_per_launch": alg_bytes,
                     "traffic": traffic,
                     # the same bytes over the time of a call that cannot overlap its neighbours
                     "frac_isolated_call": alg_bytes / (us_isolated * 1e-6) / 1e9 / peak,
                     "frac_graph_replay": (alg_bytes / (us_graph * 1e-6) / 1e9 / peak) if isinstance(us_graph, float) else None},
        "clocks": clocks,
        "e2e": {"value": us_e2e, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps,
                "what": "sparrow_verify_step_host: pinned host q / new K,V rows / parents read over the host link "
                        "by the ingest kernel every step, out + lse stored into pinned host memory by the attention "
                        "kernel, stream synchronised every step (latency policy); the committed KV prefix stays resident"},
        "gpu_launches": launches_timed,
    }
    if rank == 0 and not args.no_cpu_baseline and world == 1:
        us_cpu, cores, reps = oracle_time_c2()
        line["cpu_baseline"] = {"value": us_cpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{reps} full C2 calls (448 (token, head) rows x 26,128 keys each)"}
    elif rank == 0:
        line["cpu_baseline"] = None

    if not args.headline_only and rank == 0 and world == 1:
        del cases, batch, outs, lses, warm
        torch.cuda.empty_cache()
        line["other_configs"] = extra_configs(W, B, torch, dev, l2, peak, peaks, args.all_configs)

    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_only(args, W, B, torch, dev, l2, steps, warmup):
    """One configuration, one policy, few calls: what a profiler capture runs."""
    if args.only == "HSR":
        d_model, m_tok, n_w = 3584, 48, 12
        ws_ = [(W.normal_bf16(W.config_seed(5, r), 63, (d_model, 2 * d_model), dev).float() / (2 * d_model) ** 0.5).to(torch.bfloat16)
               for r in range(n_w)]
        e_ = W.normal_bf16(W.config_seed(5), 61, (m_tok, d_model), dev)
        h_ = W.normal_bf16(W.config_seed(5), 62, (m_tok, d_model), dev)
        z_ = torch.empty((m_tok, d_model), dtype=torch.bfloat16, device=dev)
        hctx = B.Context.for_cache(torch.empty((1, W.HKV, 128, W.D), dtype=torch.bfloat16, device=dev), W.SCALE)

        def run(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(); e0.record()
            for i in range(n):
                B.sparrow_hsr_fuse(hctx, e_, h_, ws_[i % n_w], None, z_)
            e1.record(); torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / n
        run(warmup)
        us = run(steps)
        by = d_model * 2 * d_model * 2 + 3 * m_tok * d_model * 2
        print(json.dumps({"only": "HSR", "workload": f"z = FC(e (+) h), {m_tok} tokens, d = {d_model}", "steps": steps, "warmup": warmup,
                          "us_per_call_from_python": us, "algorithmic_bytes_per_call": by, "rotation": n_w,
                          "device_status": hctx.last_device_status()}), flush=True)
        return
    ci = {"C1": 0, "C2": 1, "C3": 2, "C5": 4}[args.only]
    probe = W.make_config(ci, "cpu")
    n_caches = 3 if ci == 4 else max(4, -(-4 * l2 // probe.kv_bytes()))
    cases, ctx, outs, lses, batch = build_rotation(W, B, torch, dev, ci, n_caches, calls_per_batch=max(n_caches, min(1000, steps)))
    ctx.set_plan_policy({"latency": B.PLAN_LATENCY, "balanced": B.PLAN_BALANCED, "throughput": B.PLAN_THROUGHPUT}[args.policy])
    if args.single_calls:
        singles = [B.VerifyBatch([(c.q, c.k, c.v, c.kv_len, c.parents, c.T, o, l)]) for c, o, l in zip(cases, outs, lses)]

        def run(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(); e0.record()
            for i in range(n):
                B.sparrow_verify_attn_batch(ctx, singles[i % len(singles)])
            e1.record(); torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / n
        run(warmup)
        us = run(steps)
    else:
        time_calls(ctx, batch, warmup, B, torch)
        us = time_calls(ctx, batch, steps, B, torch)
    by = probe.kv_bytes() + probe.io_bytes()
    print(json.dumps({"only": args.only, "workload": probe.name, "plan_policy": args.policy, "single_calls": bool(args.single_calls),
                      "steps": steps, "warmup": warmup, "us_per_call": us, "algorithmic_bytes_per_call": by,
                      "hbm_gbs": by / us / 1e3, "tflops": probe.flops() / us / 1e6, "rotation": n_caches,
                      "target_items": ctx.plan_target_items(), "device_status": ctx.last_device_status()}), flush=True)


def POLICIES(B):
    return (("throughput", B.PLAN_THROUGHPUT), ("balanced", B.PLAN_BALANCED), ("latency", B.PLAN_LATENCY))


def extra_configs(W, B, torch, dev, l2, peak, peaks, anchored_variants):
    """Times C1, C3, C4 and the 28-layer C5 step (same timing rules as the headline: rotation over
    caches larger than 4 x L2, CUDA events, calls enqueued from C).  Returns a list of records;
    each is also printed on stderr as it is finished."""
    results = []
    tf_peak = peaks.get("bf16_tflops_sustained")

    def emit(d):
        results.append(d)
        print(json.dumps(d), file=sys.stderr, flush=True)

    for ci, name in ((0, "C1"), (2, "C3")):
        probe = W.make_config(ci, "cpu")
        n_caches = max(4, -(-4 * l2 // probe.kv_bytes()))
        cases, ctx, outs, lses, batch = build_rotation(W, B, torch, dev, ci, n_caches)
        by = probe.kv_bytes() + probe.io_bytes()
        for pname, pol in POLICIES(B):
            ctx.set_plan_policy(pol)
            time_calls(ctx, batch, 1000, B, torch)
            us = time_calls(ctx, batch, 20000, B, torch)
            iso = time_isolated_calls(ctx, cases, outs, lses, 200, B, torch)
            emit({"config": name, "workload": probe.name, "plan_policy": pname, "us_per_call": us, "hbm_gbs": by / us / 1e3,
                  "frac_of_measured_hbm": by / us / 1e3 / peak, "tflops": probe.flops() / us / 1e6,
                  "frac_of_bf16_sustained": (probe.flops() / us / 1e6 / tf_peak) if tf_peak else None,
                  "us_per_call_isolated": iso, "frac_of_measured_hbm_isolated": by / iso / 1e3 / peak,
                  "algorithmic_bytes": by, "rotation": n_caches})
        del cases, ctx, outs, lses, batch
        torch.cuda.empty_cache()
    # C4: anchored mode, rotate over full-length buffers
    ac = [W.make_config(3, dev, layer=r) for r in range(8)]
    actx = B.Context.for_cache(ac[0].k, W.SCALE)
    aout = torch.empty_like(ac[0].q)
    alse = torch.empty((1, W.HQ, ac[0].T), dtype=torch.float32, device=dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def anchor_loop(n):
        for i in range(n):
            c = ac[i % len(ac)]
            B.sparrow_anchor_attn(actx, c.q, c.k, c.v, c.anchor_idx, c.n_anchor, c.window, c.T, aout, alse)
    anchor_loop(200)
    torch.cuda.synchronize(); ev0.record(); anchor_loop(3000); ev1.record(); torch.cuda.synchronize()
    us_python = ev0.elapsed_time(ev1) * 1e3 / 3000
    # the same calls replayed from a CUDA graph: what the GPU needs when the host is out of the way
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        for i in range(8):
            c = ac[i % len(ac)]
            B.sparrow_anchor_attn(actx, c.q, c.k, c.v, c.anchor_idx, c.n_anchor, c.window, c.T, aout, alse, stream=side)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for i in range(64):
                c = ac[i % len(ac)]
                B.sparrow_anchor_attn(actx, c.q, c.k, c.v, c.anchor_idx, c.n_anchor, c.window, c.T, aout, alse, stream=side)
        graph.replay(); side.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(side)
        for _ in range(50):
            graph.replay()
        g1.record(side); side.synchronize()
    emit({"config": "C4", "workload": ac[0].name, "us_per_call": g0.elapsed_time(g1) * 1e3 / (50 * 64),
          "us_per_call_from_python": us_python, "gathered_bytes": ac[0].kv_bytes(),
          "note": "gather kernel on the full-length cache; latency-bound; us_per_call = 64 calls replayed from a CUDA graph, "
                  "the other figure one Python call each"})
    del graph
    # the same rows on a compacted cache: gathered once, then a contiguous stream for the tensor-core kernel
    cap_c = ac[0].n_anchor
    kc = [torch.empty((1, W.HKV, cap_c, W.D), dtype=torch.bfloat16, device=dev) for _ in ac]
    vc = [torch.empty_like(x) for x in kc]
    for c, kk, vv in zip(ac, kc, vc):
        B.sparrow_compact_anchors(actx, c.k, c.v, c.anchor_idx, c.n_anchor, kk, vv, cap_c, 0)
    cctx = B.Context.for_cache(kc[0], W.SCALE)
    cctx.set_plan_policy(B.PLAN_LATENCY)
    chain = torch.arange(-1, ac[0].T - 1, dtype=torch.int32, device=dev)[None].contiguous()
    cbatch = B.VerifyBatch([(c.q, kk, vv, [c.n_anchor - c.T], chain, c.T, aout, alse) for c, kk, vv in zip(ac, kc, vc)] * 100)
    time_calls(cctx, cbatch, 800, B, torch)
    singles_c = [type("C", (), dict(q=c.q, k=kk, v=vv, kv_len=[c.n_anchor - c.T], parents=chain, T=c.T)) for c, kk, vv in zip(ac, kc, vc)]
    emit({"config": "C4-compact", "workload": "C4 on the compacted anchor rows (sparrow_compact_anchors once, then sparrow_verify_attn)",
          "us_per_call": time_calls(cctx, cbatch, 8000, B, torch),
          "us_per_call_isolated": time_isolated_calls(cctx, singles_c, [aout] * len(ac), [alse] * len(ac), 200, B, torch),
          "note": "enqueued from C; contiguous TMA stream, no gather"})
    del kc, vc, cctx, cbatch
    if anchored_variants:
        # the same anchors with a 32-node draft tree behind them, queries = its last 8 nodes
        T_tree, T_new = 32, 8
        tc_ = [W.make_anchor_case(W.config_seed(3, 100 + r), W.c4_anchor_list(T_tree), W.C4_WINDOW, T_tree, 1, dev) for r in range(8)]
        par = torch.tensor([W.random_tree_parents(W.config_seed(3, 0), 77, T_tree)], dtype=torch.int32, device=dev)
        tctx = B.Context.for_cache(tc_[0].k, W.SCALE)
        tq = [c.q[:, T_tree - T_new:].contiguous() for c in tc_]
        tout = torch.empty_like(tq[0])
        tlse = torch.empty((1, W.HQ, T_new), dtype=torch.float32, device=dev)

        def tree_loop(n):
            for i in range(n):
                c = tc_[i % len(tc_)]
                B.sparrow_anchor_attn_tree(tctx, tq[i % len(tc_)], c.k, c.v, c.anchor_idx, c.n_anchor, c.window, par,
                                           T_tree, T_new, tout, tlse)
        tree_loop(200)
        torch.cuda.synchronize(); ev0.record(); tree_loop(3000); ev1.record(); torch.cuda.synchronize()
        emit({"config": "C4-tree", "workload": "anchored, 448 text anchors + 32-node draft tree, 8 query nodes",
              "us_per_call": ev0.elapsed_time(ev1) * 1e3 / 3000, "note": "launched from Python; latency-bound"})
        del tc_, tctx
    del ac, actx
    torch.cuda.empty_cache()
    # Draft-model input fusion z = FC(e (+) h) (Eq. 1) at a Qwen2-7B-like width: a weight-streaming GEMM,
    # rotated over enough weight matrices to stay out of L2, replayed from a CUDA graph (the call
    # encodes three tensor maps on the host, which a per-call launch loop would be timing instead)
    d_model, m_tok = 3584, 48
    n_w = max(4, -(-4 * l2 // (d_model * 2 * d_model * 2)))
    ws_ = [(W.normal_bf16(W.config_seed(5, r), 63, (d_model, 2 * d_model), dev).float() / (2 * d_model) ** 0.5).to(torch.bfloat16)
           for r in range(n_w)]
    e_ = W.normal_bf16(W.config_seed(5), 61, (m_tok, d_model), dev)
    h_ = W.normal_bf16(W.config_seed(5), 62, (m_tok, d_model), dev)
    b_ = W.normal_bf16(W.config_seed(5), 64, (d_model,), dev)
    z_ = torch.empty((m_tok, d_model), dtype=torch.bfloat16, device=dev)
    hk = torch.empty((1, W.HKV, 128, W.D), dtype=torch.bfloat16, device=dev)
    hctx = B.Context.for_cache(hk, W.SCALE)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        for w_ in ws_:
            B.sparrow_hsr_fuse(hctx, e_, h_, w_, b_, z_, stream=side)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for w_ in ws_:
                B.sparrow_hsr_fuse(hctx, e_, h_, w_, b_, z_, stream=side)
        graph.replay(); side.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(side)
        for _ in range(100):
            graph.replay()
        g1.record(side); side.synchronize()
    us = g0.elapsed_time(g1) * 1e3 / (100 * n_w)
    by = d_model * 2 * d_model * 2 + 2 * m_tok * d_model * 2 + d_model * 2 + m_tok * d_model * 2
    emit({"config": "HSR", "workload": f"z = FC(e (+) h), {m_tok} tokens, d = {d_model} (weights {d_model} x {2 * d_model} bf16)",
          "us_per_call": us, "algorithmic_bytes": by, "hbm_gbs": by / us / 1e3, "frac_of_measured_hbm": by / us / 1e3 / peak,
          "rotation": n_w, "device_status": hctx.last_device_status(),
          "note": "rotation over weight matrices larger than 4 x L2, calls replayed from a CUDA graph"})
    del graph, ws_, hctx
    torch.cuda.empty_cache()
    # C5: 28 layers, each with its own cache (about 15 GB resident)
    layers = [W.make_config(4, dev, layer=l) for l in range(28)]
    ctx = B.Context.for_cache(layers[0].k, W.SCALE)
    outs = [torch.empty_like(c.q) for c in layers]
    lses = [torch.empty((c.B, W.HQ, c.T), dtype=torch.float32, device=dev) for c in layers]
    batch = B.VerifyBatch([(c.q, c.k, c.v, c.kv_len, c.parents, c.T, o, l) for c, o, l in zip(layers, outs, lses)] * 10)
    by = sum(c.kv_bytes() + c.io_bytes() for c in layers)
    fl = sum(c.flops() for c in layers)
    for pname, pol in POLICIES(B):
        ctx.set_plan_policy(pol)
        time_calls(ctx, batch, 28 * 5, B, torch)
        us = time_calls(ctx, batch, 28 * 50, B, torch)
        emit({"config": "C5", "workload": "batch 8 ragged, T=32 tree, 28 layers per step", "plan_policy": pname,
              "us_per_step": us * 28, "us_per_layer": us, "hbm_gbs": by / (us * 28) / 1e3,
              "frac_of_measured_hbm": by / (us * 28) / 1e3 / peak, "tflops": fl / (us * 28) / 1e6,
              "frac_of_bf16_sustained": (fl / (us * 28) / 1e6 / tf_peak) if tf_peak else None,
              "us_per_layer_isolated": time_isolated_calls(ctx, layers, outs, lses, 56, B, torch),
              "algorithmic_bytes_per_step": by, "kv_len": layers[0].kv_len})
    return results


if __name__ == "__main__":
    main()
