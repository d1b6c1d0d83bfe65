"""Where the time of one call goes: builds the library with -DSPARROW_TIMELINE (a copy next to the
shipped one, never loaded by anything else), runs isolated calls and prints, per phase, when the
first, the median and the last CTA reached it (%globaltimer, microseconds after the stream
position just before the call).

    python -m paper_2602_15318_b200.timeline --config C2 --policy latency
    python -m paper_2602_15318_b200.timeline --config C2 --policy throughput --burst 20
    python -m paper_2602_15318_b200.timeline --hsr

With --burst N the N calls are enqueued back to back from C (one sparrow_verify_attn_batch, as the
bench's timed region does) and one line per call says when its CTAs started, left their main loop,
stored their partial rows and when its merged rows were written.

Stamping costs a few stores per CTA; the figures are for reading the shape of a call, the bench
times the shipped library.
"""
import argparse
import ctypes
import os
import subprocess

import numpy as np
import torch

from . import binding as B
from . import build as _build
from . import workloads as W

LIB = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsparrow_attn_timeline.so")
CALLS, CTAS, SLOTS = 32, 256, 16

VERIFY_SLOTS = ["kernel entered", "set-up done (barriers, TMEM)", "Q landed", "first K tile landed",
                "last product issued", "softmax loop left", "last product complete", "partial rows stored",
                "finisher: all arrivals seen", "finisher: previous call done", "finisher: merged rows written",
                "leaving", "finisher: bulk copies issued", "finisher: pieces folded", "finisher: groups reduced",
                "finisher: bulk copies landed"]
HSR_SLOTS = ["kernel entered", "set-up done (barriers, TMEM)", "first tile landed", "last MMA issued",
             "accumulator complete", "partial sums pushed", "cluster barrier passed", "z written, leaving"]


def build_timeline_library() -> str:
    if os.path.exists(LIB) and os.path.getmtime(LIB) >= _build._newest_source():
        return LIB
    cmd = [_build.nvcc()] + _build.NVCC_FLAGS + ["-DSPARROW_TIMELINE", "-I" + os.path.join(_build.ROOT, "include"),
                                                  "-I" + _build.CSRC, "-o", LIB] + _build.SOURCES + ["-lcuda"]
    subprocess.run(cmd, check=True)
    return LIB


def _table(rows, names):
    """rows: list of [n_cta, SLOTS] arrays of ns relative to the mark (-1 = slot not reached)."""
    print(f"{'phase':40s} {'first':>8s} {'median':>8s} {'last':>8s}   (us, medians over {len(rows)} calls)")
    for k, name in enumerate(names):
        first, med, last = [], [], []
        for rel in rows:
            c = rel[:, k]
            c = c[c >= 0]
            if len(c):
                first.append(c.min()); med.append(np.median(c)); last.append(c.max())
        if first:
            print(f"{name:40s} {np.median(first) / 1e3:8.2f} {np.median(med) / 1e3:8.2f} {np.median(last) / 1e3:8.2f}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", choices=["C1", "C2", "C3", "C5"], default="C2")
    ap.add_argument("--policy", choices=["latency", "balanced", "throughput"], default="latency")
    ap.add_argument("--hsr", action="store_true", help="the Eq. 1 projection (48 tokens, d = 3584) instead of attention")
    ap.add_argument("--calls", type=int, default=40)
    ap.add_argument("--burst", type=int, default=0, help="enqueue this many calls (at most 32) back to back and print one line per call")
    args = ap.parse_args()

    B.LIB_PATH = build_timeline_library()
    L = B.lib()
    L.sparrow_timeline_read.argtypes = [ctypes.c_void_p]
    L.sparrow_timeline_mark.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    dev = "cuda:0"
    torch.cuda.set_device(0)
    marks = torch.zeros(2, dtype=torch.int64, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    n_rot = 6

    if args.hsr:
        d, M = 3584, 48
        ws = [(W.normal_bf16(100 + r, 63, (d, 2 * d), dev).float() / (2 * d) ** 0.5).to(torch.bfloat16) for r in range(n_rot)]
        e, h = W.normal_bf16(1, 61, (M, d), dev), W.normal_bf16(1, 62, (M, d), dev)
        z = torch.empty((M, d), dtype=torch.bfloat16, device=dev)
        ctx = B.Context.for_cache(torch.empty((1, W.HKV, 128, W.D), dtype=torch.bfloat16, device=dev), W.SCALE)
        call = lambda i: B.sparrow_hsr_fuse(ctx, e, h, ws[i % n_rot], None, z)
        names, what = HSR_SLOTS, "sparrow_hsr_fuse, 48 tokens, 3584 x 7168 weights"
    else:
        cfg = int(args.config[1]) - 1                      # workloads.make_config counts from 0
        cases = [W.make_config(cfg, dev, layer=r) for r in range(n_rot)]
        ctx = B.Context.for_cache(cases[0].k, W.SCALE)
        ctx.set_plan_policy({"latency": B.PLAN_LATENCY, "balanced": B.PLAN_BALANCED, "throughput": B.PLAN_THROUGHPUT}[args.policy])
        outs = [torch.empty_like(c.q) for c in cases]
        lses = [torch.empty((c.B, W.HQ, c.T), dtype=torch.float32, device=dev) for c in cases]

        def call(i):
            c = cases[i % n_rot]
            B.sparrow_verify_attn(ctx, c.q, c.k, c.v, c.kv_len, c.parents, c.T, outs[i % n_rot], lses[i % n_rot])
        names, what = VERIFY_SLOTS, f"sparrow_verify_attn, {args.config}, {args.policy} policy"

    def read_table():
        buf = np.zeros(CALLS * CTAS * SLOTS, dtype=np.uint64)
        if L.sparrow_timeline_read(buf.ctypes.data) != 0:
            raise SystemExit("reading the stamp table failed")
        return buf.reshape(CALLS, CTAS, SLOTS).astype(np.int64)

    if args.burst:
        if args.hsr or not 1 <= args.burst <= CALLS:
            raise SystemExit("--burst: 1 .. 32 attention calls")
        n = args.burst
        batch = B.VerifyBatch([(cases[i % n_rot].q, cases[i % n_rot].k, cases[i % n_rot].v, cases[i % n_rot].kv_len,
                                cases[i % n_rot].parents, cases[i % n_rot].T, outs[i % n_rot], lses[i % n_rot]) for i in range(n)])
        runs = []
        for rep in range(8):
            torch.cuda.synchronize()
            L.sparrow_timeline_clear()
            torch.cuda._sleep(400000)
            L.sparrow_timeline_mark(marks.data_ptr(), stream)
            B.sparrow_verify_attn_batch(ctx, batch)
            L.sparrow_timeline_mark(marks.data_ptr() + 8, stream)
            torch.cuda.synchronize()
            if ctx.last_device_status() != 0:
                raise SystemExit("device status set")
            t = read_table()
            m0, m1 = int(marks[0]), int(marks[1])
            used = [c for c in range(CALLS) if (t[c, :, 0] > 0).any()]
            used.sort(key=lambda c: t[c, :, 0][t[c, :, 0] > 0].min())
            per_call = []
            for c in used:
                tc = t[c][t[c, :, 0] > 0]
                rel = np.where(tc > 0, tc - m0, -1)
                col = lambda k, f: (f(rel[:, k][rel[:, k] >= 0]) / 1e3 if (rel[:, k] >= 0).any() else float("nan"))
                per_call.append((rel.shape[0], col(0, np.min), col(0, np.max), col(5, np.min), col(5, np.max), col(7, np.max),
                                 col(8, np.min), col(10, np.max), col(11, np.max)))
            runs.append(((m1 - m0) / 1e3, per_call))
        runs = runs[2:]
        print(f"{what}: burst of {n} calls; mark before -> mark after: {np.median([r[0] for r in runs]):.1f} us "
              f"({np.median([r[0] for r in runs]) / n:.2f} us per call); medians over {len(runs)} bursts, us after the first mark")
        print(f"{'call':>4s} {'CTAs':>5s} {'first in':>9s} {'last in':>9s} {'loop left: first':>17s} {'last':>8s} {'stored':>8s} "
              f"{'arrivals seen':>14s} {'merged':>8s} {'last out':>9s}")
        for i in range(len(runs[0][1])):
            vals = np.median(np.array([r[1][i] for r in runs if len(r[1]) > i], dtype=np.float64), axis=0)
            print(f"{i:4d} {int(vals[0]):5d} {vals[1]:9.1f} {vals[2]:9.1f} {vals[3]:17.1f} {vals[4]:8.1f} {vals[5]:8.1f} {vals[6]:14.1f} {vals[7]:8.1f} {vals[8]:9.1f}")
        return

    rows, spans = [], []
    for i in range(args.calls):
        torch.cuda.synchronize()
        L.sparrow_timeline_clear()
        torch.cuda._sleep(200000)                      # the host runs ahead: its launch latency is not in the picture
        L.sparrow_timeline_mark(marks.data_ptr(), stream)
        call(i)
        L.sparrow_timeline_mark(marks.data_ptr() + 8, stream)
        torch.cuda.synchronize()
        if ctx.last_device_status() != 0:
            raise SystemExit("device status set")
        t = read_table().reshape(CALLS * CTAS, SLOTS)
        t = t[t[:, 0] > 0]
        m0, m1 = int(marks[0]), int(marks[1])
        rows.append(np.where(t > 0, t - m0, -1))
        spans.append(m1 - m0)
    rows, spans = rows[args.calls // 4:], spans[args.calls // 4:]
    print(f"{what}: {rows[0].shape[0]} CTAs; mark before the call -> mark after it: {np.median(spans) / 1e3:.2f} us")
    _table(rows, names)

if __name__ == "__main__":
    main()
