"""Phase tables of the one-launch inner loop and of the streaming worker kernel, from %globaltimer stamps.

    python -m paper_1901_08924_b200.trace [--workload ls|alpc] [--bits B] [--rows N] [--steps M]
    python -m paper_1901_08924_b200.trace --workload stream [--batch B] [--bits B] [--rows N]

Profilers cannot replay the cooperative cluster launch of the one-launch loop, so its time is accounted for with
time stamps instead: the library is built a second time with -DLPC_TRACE (liblpcsvrg_trace.so, see build.py), in which
thread 0 of CTA (0, 0) stores %globaltimer at every phase boundary of steps 8..71 of a launch.  This module runs a
workload on that build and prints the median duration of every phase.  The stamped build runs several per cent slower
than the plain one and the timer has a grain of 32 ns: read the table for where the time goes, not for the total.

workloads (synthetic, shapes of the benchmark's):
  ls    least squares, d = 4,096, N = 16 workers, B = 8, b = 4, clip 3 std   (Algorithm 1)
  alpc  logistic, d = 8,192, ill-conditioned columns, N = 32, B = 16, b = 2 (or --bits 8), clip 2 std   (Algorithm 2)
  stream  the fused worker kernel on large minibatches: logistic, 65,536 x 8,192, N = 32, B = 256 (or --batch 1024) rows per
          worker, b = 2.  In the stamped build thread 0 of EVERY CTA stores %globaltimer at six points of the kernel; the
          table gives the spread of each point over the 128 CTAs of one launch, next to the launch's CUDA-event time.
"""
import argparse
import ctypes as C
import os
import statistics
import sys

PHASES = [
    (0, 1, "rounding bits (Philox)"),
    (1, 2, "sampling of the next step's rows"),
    (2, 3, "loads of all workers' words issued -> all tags valid (the next step's row copies are issued meanwhile)"),
    (3, 4, "decode + average + proximal step (Algorithm 2: y, z updates and coupling)"),
    (4, 5, "wait for this step's rows"),
    (5, 6, "margins (partial sums, warp reduction, block barrier)"),
    (6, 7, "cluster exchange of the margin partial sums"),
    (7, 8, "coefficients + block barrier"),
    (8, 9, "u"),
    (9, 10, "statistics of u (warp reductions, block barrier)"),
    (10, 11, "block statistics + issue of the remaining row fetches"),
    (11, 12, "cluster exchange of the statistics + scale (Eq. 2) + block barrier"),
    (12, 13, "quantize + pack + store the tagged words"),
    (13, 14, "end of step"),
]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="ls", choices=["ls", "alpc", "stream"])
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--bits", type=int, default=0)
    ap.add_argument("--rows", type=int, default=0)
    ap.add_argument("--steps", type=int, default=128)
    args = ap.parse_args()

    from . import build
    os.environ["LPC_LIBRARY"] = build.build(trace=True)
    import torch
    from . import lpc, synth
    assert lpc.LIB_PATH == os.environ["LPC_LIBRARY"], "import this module before paper_1901_08924_b200.lpc"

    dev = torch.device("cuda", 0)
    if args.workload == "stream":
        return stream_table(args, dev, torch, lpc, synth)
    if args.workload == "ls":
        n, d, N, B, b = args.rows or 16384, 4096, 16, 8, args.bits or 4
        X, y, _ = synth.linear_problem(n, d, loss="least_squares", sparsity=0.05, noise=0.01, seed=0, device=dev)
        ctx = lpc.Context(X, y, lpc.LEAST_SQUARES, 1e-4, N, B, b, lpc.CLIP_STD, 3.0, 0)
        L = float((X.double() ** 2).sum(dim=1).max().item())
        run = lambda k0: ctx.inner_steps(1.0 / (6.0 * L), k0, args.steps)
        info = (lpc.INFO_LOOP_CLUSTER_SIZE, lpc.INFO_LOOP_ROW_SLOTS, lpc.INFO_LOOP_COORDS_PER_THREAD)
    else:
        n, d, N, B, b = args.rows or 32768, 8192, 32, 16, args.bits or 2
        X, y, _ = synth.linear_problem(n, d, loss="logistic", sparsity=0.02, noise=0.1, seed=1, col_scale_range=(0.1, 10.0),
                                       device=dev)
        ctx = lpc.Context(X, y, lpc.LOGISTIC, 1e-5, N, B, b, lpc.CLIP_STD, 2.0, 0)
        L = 0.25 * float((X * X).sum(dim=1).max().item())
        ctx.alpc_begin()
        run = lambda k0: ctx.alpc_double_sample_steps(0.5, 0.5, 1.0 / (3.0 * L), 1.0 / (4.0 * L), k0, args.steps)
        info = (lpc.INFO_ALPC_LOOP_CLUSTER_SIZE, lpc.INFO_ALPC_LOOP_ROW_SLOTS, lpc.INFO_ALPC_LOOP_COORDS_PER_THREAD)
    ctx.snapshot_full_grad()
    st = torch.cuda.current_stream(dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    run(0)
    ctx.sync_status()
    ev[0].record(st)
    run(args.steps)
    ev[1].record(st)
    ctx.sync_status()
    assert ctx.query(lpc.INFO_LOOP_LAUNCHES) == 2, "the one-launch loop did not run"
    buf = (C.c_ulonglong * (64 * 16))()
    read = lpc.lib().lpc_trace_read
    read.restype, read.argtypes = C.c_int, [C.POINTER(C.c_ulonglong)]
    assert read(buf) == 0
    steps = min(64, args.steps - 8)
    marks = [[buf[s * 16 + i] for i in range(16)] for s in range(steps)]
    cs, slots, ept = (ctx.query(i) for i in info)
    print("workload %s: n = %d, d = %d, N = %d, B = %d, b = %d; cluster size %d, %d row slots, %d coordinates per thread"
          % (args.workload, n, d, N, B, b, cs, slots, ept))
    print("CUDA events: %.3f us per step over %d steps (stamped build)" % (ev[0].elapsed_time(ev[1]) * 1e3 / args.steps, args.steps))
    print("| phase (thread 0 of CTA (0,0), median over %d steps) | ns |" % steps)
    print("|---|---|")
    total = 0
    for a, b_, name in PHASES:
        v = [m[b_] - m[a] for m in marks if m[a] and m[b_] and m[b_] >= m[a]]
        med = statistics.median(v) if v else float("nan")
        total += med if v else 0
        print("| %s | %.0f |" % (name, med))
    period = [marks[s + 1][0] - marks[s][0] for s in range(steps - 1)]
    print("| step period | %.0f |" % statistics.median(period))
    print("| looks at the words until all tags matched (median, max) | %d, %d |"
          % (statistics.median(m[15] for m in marks), max(m[15] for m in marks)))
    ctx.close()


STREAM_MARKS = [(0, "kernel entry"), (2, "first bulk copies issued (by the refill warp)"),
                (1, "block-wide prologue done (sampling of the whole batch, barrier set-up, cluster arrival)"),
                (3, "every CTA of the cluster has started"), (5, "last group added to u, u with the owners of its coordinates"),
                (6, "scale known (statistics, exchange across the cluster, Eq. 2)"), (7, "codes stored")]


def stream_table(args, dev, torch, lpc, synth):
    n, d, N, B, b = args.rows or 65536, 8192, 32, args.batch, args.bits or 2
    X, y, _ = synth.linear_problem(n, d, loss="logistic", sparsity=0.02, noise=0.1, seed=1, col_scale_range=(0.1, 10.0),
                                   device=dev)
    ctx = lpc.Context(X, y, lpc.LOGISTIC, 1e-5, N, B, b, lpc.CLIP_STD, 2.0, 0)
    ctx.snapshot_full_grad()
    ctx.inner_steps(1e-3, 0, 5)
    ctx.set_option(lpc.OPT_PROFILE, 1)
    ctx.inner_steps(1e-3, 5, 10)
    ctx.sync_status()
    prof = ctx.get_profile()
    cs = ctx.query(lpc.INFO_STEP_CLUSTER_SIZE)
    ctas = N * cs
    buf = (C.c_ulonglong * (1024 * 8))()
    read = lpc.lib().lpc_debug_stream_trace
    read.restype, read.argtypes = C.c_int, [C.POINTER(C.c_ulonglong)]
    assert read(buf) == 0
    marks = [[buf[c * 8 + i] for i in range(8)] for c in range(ctas)]
    t0 = min(m[0] for m in marks)
    print("workload stream: n = %d, d = %d, N = %d, B = %d, b = %d; clusters of %d CTAs, ring of %d stages"
          % (n, d, N, B, b, cs, ctx.query(lpc.INFO_STEP_RING_STAGES)))
    print("CUDA events around one launch: %.2f us (stamped build, average of 10)" % (prof["worker"][0] / prof["worker"][1] * 1e3))
    print("| mark (thread 0 of each of the %d CTAs of the last launch, ns from the first CTA's entry) | min | median | max |" % ctas)
    print("|---|---|---|---|")
    for i, name in STREAM_MARKS:
        v = sorted(m[i] - t0 for m in marks)
        print("| %s | %d | %d | %d |" % (name, v[0], v[len(v) // 2], v[-1]))
    ctx.close()


if __name__ == "__main__":
    sys.exit(main())
