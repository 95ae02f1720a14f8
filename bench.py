#!/usr/bin/env python
"""Benchmark of the LPC-SVRG hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one LPC-SVRG epoch of the least-squares + L1 workload (131,072 x 4,096, 16 workers,
minibatch 8, 4 bits, clip 3 std): the snapshot full-gradient pass over X followed by m = n/(8N) =
1,024 fused inner iterations.  The headline value is inner iterations per second over all GPUs
(each GPU runs an independent replica: the method's communication is counted, never sent).
The JSON line also carries the roofline of the dominant kernel, per-kernel device times, the
stand-alone quantize+aggregate bandwidths, the end-to-end number from host buffers and the CPU
oracle's throughput on the same workload.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "svrg_inner_iters_per_sec"
UNIT = "inner-iters/s"

WORKLOADS = {
    # name: n, d, loss, lambda_l1, N, B, b, clip c (std rule), sparsity of w*, label noise
    "lpc_svrg_ls_131072x4096_N16_B8_b4": dict(n=131072, d=4096, loss="least_squares", lam=1e-4, N=16, B=8, b=4, c=3.0,
                                              sparsity=0.05, noise=0.01),
    # the main workload with 1/8 of the rows (X = 268 MB, still larger than L2): for profiler captures
    "lpc_svrg_ls_16384x4096_N16_B8_b4": dict(n=16384, d=4096, loss="least_squares", lam=1e-4, N=16, B=8, b=4, c=3.0,
                                             sparsity=0.05, noise=0.01),
    "lpc_svrg_logistic_4000x1000_N4_B1_b2": dict(n=4000, d=1000, loss="logistic", lam=1e-4, N=4, B=1, b=2, c=2.5,
                                                 sparsity=0.10, noise=0.1, m=1000, eta=0.1),
}
DEFAULT_WORKLOAD = "lpc_svrg_ls_131072x4096_N16_B8_b4"


def read_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            for line in open(self.path):
                p = [t.strip() for t in line.split(",")]
                if len(p) >= 7 and p[0].replace(".", "").isdigit():
                    rows.append(p)
            os.unlink(self.path)
        except Exception:
            pass
        if rows:
            out["sm_mhz"] = statistics.median(float(r[0]) for r in rows)
            out["sm_max_mhz"] = max(float(r[1]) for r in rows)
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            out["reasons"] = [nm for i, nm in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
            out["samples"] = len(rows)
        return out


def visible_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        parts = [p for p in vis.split(",") if p]
        if local_rank < len(parts) and parts[local_rank].isdigit():
            return int(parts[local_rank])
    return local_rank


def make_problem(w, seed, device):
    import torch
    from paper_1901_08924_b200 import synth
    X, y, _ = synth.linear_problem(w["n"], w["d"], loss=w["loss"], sparsity=w["sparsity"], noise=w["noise"], seed=seed,
                                   device=device)
    m = w.get("m", w["n"] // (w["B"] * w["N"]))
    if "eta" in w:
        eta = w["eta"]
    else:  # eta = 1/(6 L) with L = c_loss * max_a ||X_a||^2 (c_loss = 1 least squares, 1/4 logistic)
        L = float((X.double() ** 2).sum(dim=1).max().item()) * (1.0 if w["loss"] == "least_squares" else 0.25)
        eta = 1.0 / (6.0 * L)
    return X, y, m, float(eta)


def loss_code(w):
    from paper_1901_08924_b200 import lpc
    return lpc.LEAST_SQUARES if w["loss"] == "least_squares" else lpc.LOGISTIC


def bytes_per_launch(w, m):
    """Algorithmic bytes one launch of each kernel class must move."""
    n, d, N, B, b = w["n"], w["d"], w["N"], w["B"], w["b"]
    W = (d * b + 31) // 32
    return {
        "snapshot": n * d * 4 + n * 4 + n * 4 + d * 4,                       # X once, y, margins written, x~
        "worker": N * B * d * 4 + N * B * 8 + d * 4 + N * (W * 4 + 4),       # rows once, y + cached margin, x, codes out
        "aggregate": N * (W * 4 + 4) + 3 * d * 4,                            # codes in, mu, x in, x out
    }


def run_ours(args):
    import torch
    from paper_1901_08924_b200 import dist_util, lpc, synth

    size, rank, local = dist_util.world()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist_util.init("nccl")
    w = WORKLOADS[args.workload]
    X, y, m, eta = make_problem(w, seed=rank, device=dev)
    n, d, N, B, b = w["n"], w["d"], w["N"], w["B"], w["b"]
    ctx = lpc.Context(X, y, loss_code(w), w["lam"], N, B, b, lpc.CLIP_STD, w["c"], seed=rank)
    if args.per_step_kernels:
        ctx.set_option(lpc.OPT_PERSISTENT, 0)
    if args.loop_not_cooperative:
        ctx.set_option(lpc.OPT_LOOP_COOPERATIVE, 0)

    def epoch(s):
        ctx.snapshot_full_grad()
        ctx.inner_steps(eta, s * m, m)

    s_next = 0
    for _ in range(max(args.warmup, 3)):
        epoch(s_next)
        s_next += 1
    ctx.sync_status()
    sampler = ClockSampler(visible_index(local))
    sampler.start()
    time.sleep(0.3)
    st = torch.cuda.current_stream(dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.steps + 1)]
    dist_util.barrier()
    torch.cuda.synchronize(dev)
    t_wall = time.perf_counter()
    ev[0].record(st)
    for i in range(args.steps):
        ctx.snapshot_full_grad()
        ev[2 * i + 1].record(st)
        ctx.inner_steps(eta, s_next * m, m)
        ev[2 * i + 2].record(st)
        s_next += 1
    torch.cuda.synchronize(dev)
    dist_util.barrier()
    t_wall = time.perf_counter() - t_wall
    ms_local = ev[0].elapsed_time(ev[-1])
    snap_ms = sum(ev[2 * i].elapsed_time(ev[2 * i + 1]) for i in range(args.steps)) / args.steps
    inner_ms = sum(ev[2 * i + 1].elapsed_time(ev[2 * i + 2]) for i in range(args.steps)) / args.steps
    # keep the GPU busy a little longer so that the clock samples cover load, then stop sampling
    clocks = sampler.stop()
    ctx.sync_status()
    value, ms = dist_util.whole_job_throughput(args.steps * m, ms_local, dev)
    P_end = ctx.objective()

    # ---- per-kernel device time: the same steps again with an event pair around every launch -------------------
    ctx.set_option(lpc.OPT_PROFILE, 1)
    prof_steps = min(args.steps, 2)
    for _ in range(prof_steps):
        epoch(s_next)
        s_next += 1
    prof = ctx.get_profile()
    ctx.set_option(lpc.OPT_PROFILE, 0)
    peak, peak_kind = read_peak()
    bpl = bytes_per_launch(w, m)
    bpl["inner_loop"] = m * (bpl["worker"] + bpl["aggregate"])  # one persistent launch runs all m steps
    kernels = {}
    for name in ("snapshot", "inner_loop", "worker", "aggregate"):
        tot_ms, cnt = prof[name]
        if cnt:
            us = tot_ms / cnt * 1e3
            kernels[name] = {"launches_per_step": cnt // prof_steps, "avg_us": round(us, 3),
                             "share_of_step": round(tot_ms / prof_steps / (snap_ms + inner_ms), 4),
                             "bytes_per_launch": bpl[name], "gbs": round(bpl[name] / us * 1e-3, 1),
                             "frac": round(bpl[name] / us * 1e-3 / peak, 4)}
    dominant = max(kernels, key=lambda k: kernels[k]["avg_us"] * kernels[k]["launches_per_step"]) if kernels else None
    # Launch duration of the dominant kernel inside the timed region: the events recorded after the snapshot
    # pass and after the inner loop bracket exactly one persistent launch (or, on the per-step path, m
    # worker+aggregate pairs whose time is split by the two kernels' event-timed ratio).
    roofline = None
    if dominant:
        kd = kernels[dominant]
        if dominant == "snapshot":
            dur_us = snap_ms * 1e3
        elif dominant == "inner_loop":
            dur_us = inner_ms * 1e3
        else:
            pair = kernels["worker"]["avg_us"] + kernels["aggregate"]["avg_us"]
            dur_us = inner_ms * 1e3 / m * kd["avg_us"] / pair
        ach = kd["bytes_per_launch"] / dur_us * 1e-3
        traffic, traffic_src = None, None
        if dominant == "inner_loop":
            # profilers cannot replay the cooperative launch; the per-step worker kernel, which moves the same rows, was
            # captured instead: its DRAM bytes per step times the steps of one launch
            traffic, traffic_src = traffic_of("inner_kernel<4> (per step)", m)
            traffic_src = "taken on the per-step kernels (the one-launch loop cannot be replayed by the profiler): " + traffic_src
        elif dominant == "snapshot":
            traffic, traffic_src = traffic_of("snapshot_kernel", n * d)
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": round(ach, 1), "peak": peak, "unit": "GB/s",
                    "frac": round(ach / peak, 4), "frac_of_nominal_8TBs": round(ach / NOMINAL_HBM_GBS, 4),
                    "traffic": traffic, "traffic_source": traffic_src, "peak_source": f"of {peak_kind}",
                    "launch_us": round(dur_us, 3),
                    "note": "latency-bound: an inner step moves %.2f MB behind a strict step-to-step dependency; "
                            "kernels[] lists the bandwidth-bound kernels of the path, each with its workload"
                            % ((bpl["worker"] + bpl["aggregate"]) / 1e6),
                    "kernels": []}
        if "snapshot" in kernels:
            ks = kernels["snapshot"]
            roofline["kernels"].append(roofline_entry("snapshot_kernel", args.workload, ks["avg_us"], ks["bytes_per_launch"], peak,
                                                      "snapshot_kernel", n * d))
    launches_per_epoch = 2 + sum(kernels[k]["launches_per_step"] for k in kernels if k != "snapshot")

    out = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": size, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "step": "1 epoch = snapshot full gradient + %d inner iterations" % m,
                   "n": n, "d": d, "N": N, "B": B, "b": b, "clip": "%.1f*std" % w["c"], "eta": eta,
                   "l2": "inputs larger than L2 (X is %.2f GB, rows sampled at random)" % (n * d * 4 / 1e9),
                   "parallelism": "replicas only" if size > 1 else "1 GPU"},
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                   "samples": clocks["samples"]},
        "gpu_launches": args.steps * launches_per_epoch,
        "snapshot_ms": round(snap_ms, 4), "inner_loop_ms": round(inner_ms, 4),
        "inner_step_us": round(inner_ms * 1e3 / m, 3), "wall_s": round(t_wall, 4), "objective_end": P_end,
        "roofline": roofline, "kernels": kernels,
        "launch_plan": {"loop_cluster_size": ctx.query(lpc.INFO_LOOP_CLUSTER_SIZE),
                        "loop_coords_per_thread": ctx.query(lpc.INFO_LOOP_COORDS_PER_THREAD),
                        "loop_row_slots": ctx.query(lpc.INFO_LOOP_ROW_SLOTS),
                        "loop_launches": ctx.query(lpc.INFO_LOOP_LAUNCHES),
                        "step_cluster_size": ctx.query(lpc.INFO_STEP_CLUSTER_SIZE),
                        "snapshot_rows_per_tile": ctx.query(lpc.INFO_SNAPSHOT_ROWS_PER_TILE),
                        "snapshot_stages": ctx.query(lpc.INFO_SNAPSHOT_STAGES)},
    }
    if rank == 0 and size == 1 and not args.quick:
        out["e2e"] = e2e_bench(w, X, y, m, eta, dev)
        out["cpu_baseline"] = cpu_baseline(w, X, y, m, eta)
        del X, y
        ctx.close()
        torch.cuda.empty_cache()
        out["tiny_logistic"] = tiny_logistic_bench(dev)
        qa = quantize_aggregate_bench(dev, peak)
        roofline["kernels"] += qa.pop("roofline_kernels")
        out["quantize_aggregate"] = qa
        torch.cuda.empty_cache()
        out["alpc"] = alpc_bench(dev, peak)
        roofline["kernels"] += out["alpc"].pop("roofline_kernels")
        torch.cuda.empty_cache()
        out["fused_large_batch"] = fused_large_batch_bench(dev, peak)
        roofline["kernels"] += out["fused_large_batch"].pop("roofline_kernels")
    elif rank == 0:
        out["e2e"] = None
    ctx.close()
    dist_util.barrier()
    if rank == 0:
        print(json.dumps(out))
    dist_util.shutdown()


NOMINAL_HBM_GBS = 8000.0   # the vendor's round figure for the part's HBM3e, for context beside the measured copy rate
L2_BYTES = 126e6

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch, from the ncu captures summarised under
# profiles/: (bytes, units of that capture, summary file).  The captures are of smaller cases than the bench times
# (a few hundred MB, as profiler captures must be); traffic grows in proportion to the units a launch processes, so it
# is scaled by them.  An entry goes away when its kernel changes.
TRAFFIC = {
    "snapshot_kernel": (268.56e6 + 4.25e6, 16384 * 4096, "profiles/snapshot_kernel_ls_16384x4096.md"),
    "snapshot_kernel (logistic)": (537.00e6 + 4.16e6, 16384 * 8192, "profiles/snapshot_kernel_logistic_16384x8192.md"),
    "stats_kernel": (536.96e6 + 4.20e6, 8 * (1 << 24), "profiles/quantize_aggregate_N8_len2p24_b4_b3.md"),
    "quantize_kernel<4>": (536.95e6 + 14.21e6, 8 * (1 << 24), "profiles/quantize_aggregate_N8_len2p24_b4_b3.md"),
    "quantize_kernel<3>": (536.92e6 + 8.00e6, 8 * (1 << 24), "profiles/quantize_aggregate_N8_len2p24_b4_b3.md"),
    "unpack_average_prox_kernel<4>": (134.25e6 + 25.20e6, 1 << 24, "profiles/quantize_aggregate_N8_len2p24_b4_b3.md"),
    "unpack_average_prox_kernel<3>": (117.47e6 + 21.75e6, 1 << 24, "profiles/quantize_aggregate_N8_len2p24_b4_b3.md"),
    "code_histogram_swar_kernel<4>": (67.13e6 + 0.26e6, 8 * (1 << 24), "profiles/server_reduce4_and_code_histogram_N8_len2p24_b4.md"),
    "server_reduce4_kernel<7, sum>": (67.12e6 + 1.84e6, 1 << 24, "profiles/server_reduce4_and_code_histogram_N8_len2p24_b4.md"),
    "inner_kernel<4> (per step)": (2.220e6, 1, "profiles/inner_step_kernels_ls_16384x4096_N16_B8_b4.md"),
    "inner_kernel<2, stream>": (234.3e6 + 4.8e6, 32 * 256, "profiles/streaming_worker_kernel_logistic_16384x8192_N32_B256_b2.md"),
}


def traffic_of(name, units):
    if name not in TRAFFIC:
        return None, None
    bytes_, cap_units, src = TRAFFIC[name]
    return round(bytes_ * units / cap_units), "%s, scaled by %g" % (src, units / cap_units)


def roofline_entry(kernel, workload, avg_us, alg_bytes, peak, traffic_name=None, units=None, note=None):
    gbs = alg_bytes / avg_us * 1e-3
    tr, src = traffic_of(traffic_name, units) if traffic_name else (None, None)
    e = {"kernel": kernel, "workload": workload, "avg_us": round(avg_us, 3), "algorithmic_bytes": int(alg_bytes),
         "gbs": round(gbs, 1), "frac": round(gbs / peak, 4), "frac_of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4),
         "traffic": tr}
    if src:
        e["traffic_source"] = src
    if note:
        e["note"] = note
    return e


def _time_calls(fn, dev, reps):
    import torch
    st = torch.cuda.current_stream(dev)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        fn()
    torch.cuda.synchronize(dev)
    a.record(st)
    for _ in range(reps):
        fn()
    b.record(st)
    torch.cuda.synchronize(dev)
    return a.elapsed_time(b) / reps


def _kernel_ms(ctx, fn, reps, kinds):
    """Average device time per call of `fn`, summed over the kernel classes `kinds`, from the library's own event pair
    around every launch (the Python wrapper costs more than the short kernels)."""
    from paper_1901_08924_b200 import lpc
    for i in range(2):
        fn(i)
    ctx.sync_status()
    import torch
    ctx.set_option(lpc.OPT_PROFILE, 1)
    ctx.get_profile(reset=True)
    # the timed calls queue up behind a millisecond of busy-waiting on the stream, so that each starts when the one before
    # ends: a short kernel that finds the GPU idle is timed with the launch latency of its event pair
    torch.cuda._sleep(2_000_000)
    for i in range(reps):
        fn(2 + i)
    ctx.sync_status()
    pr = ctx.get_profile(reset=True)
    ctx.set_option(lpc.OPT_PROFILE, 0)
    return {k: pr.get(k, (0.0, 0))[0] / reps for k in kinds}


def qa_point(dev, peak, U, b, clip, reps=5):
    """Stand-alone quantize+pack then unpack+average+prox on the N vectors U (clip c*std, lambda_l1 = 1e-3, eta = 1).
    Output buffers rotate over enough sets to exceed L2, so that no call finds its own previous output there; inputs
    of at most half of L2 are reported as L2-resident, with the one-read bound of 4 + b/8 bytes per element."""
    import torch
    from paper_1901_08924_b200 import lpc
    N, ln = U.shape
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, clip, 0)
    _, stride = lpc.packed_layout(ln, b)
    out_bytes = N * stride * 4 + ln * 4
    nsets = int(max(1, min(8, -(-2 * L2_BYTES // out_bytes))))
    codes = [torch.empty((N, stride), dtype=torch.int32, device=dev) for _ in range(nsets)]
    xs = [torch.zeros(ln, device=dev) for _ in range(nsets)]
    delta = torch.empty((N, 1), dtype=torch.float32, device=dev)
    clipped = torch.empty((N, 1), dtype=torch.int32, device=dev)
    resident = N * ln * 4 <= L2_BYTES / 2
    tq = _kernel_ms(q, lambda i: q.quantize_pack(U, i, codes_out=codes[i % nsets], delta_out=delta, clipped_out=clipped),
                    reps, ("quant_stats", "other", "quant_pack", "quant_fused"))
    for c in codes[1:]:  # every set holds valid codes before the aggregator is timed
        c.copy_(codes[0])
    ta = _kernel_ms(q, lambda i: q.unpack_average_prox(codes[i % nsets], delta, ln, xs[i % nsets], 1.0, 1e-3),
                    2 * reps, ("aggregate",))["aggregate"]
    q.close()
    bq = N * ln * ((4 if resident else 8) + b / 8)
    ba = ln * (N * b / 8 + 12)
    tq_all = sum(tq.values())
    return {"N": N, "len": ln, "b": b, "clip_std": clip, "l2_resident_input": resident, "output_sets": nsets,
            "quantize_pack": {"ms": round(tq_all, 5), "stats_ms": round(tq["quant_stats"], 5), "scale_ms": round(tq["other"], 5),
                              "pack_ms": round(tq["quant_pack"], 5), "one_launch_ms": round(tq["quant_fused"], 5),
                              "bytes": bq, "gbs": round(bq / tq_all * 1e-6, 1),
                              "frac": round(bq / tq_all * 1e-6 / peak, 4), "frac_of_nominal_8TBs": round(bq / tq_all * 1e-6 / NOMINAL_HBM_GBS, 4)},
            "unpack_average_prox": {"ms": round(ta, 5), "bytes": ba, "gbs": round(ba / ta * 1e-6, 1), "frac": round(ba / ta * 1e-6 / peak, 4),
                                    "frac_of_nominal_8TBs": round(ba / ta * 1e-6 / NOMINAL_HBM_GBS, 4)},
            "combined_gbs": round((bq + ba) / (tq_all + ta) * 1e-6, 1)}


def quantize_aggregate_bench(dev, peak, log2_len=26, full=True):
    """The quantizer/aggregator sweep: N = 8 worker vectors, lengths 2^16 .. 2^28, Gaussian and Student-t (3 degrees of
    freedom) values, b in {1, 2, 3, 4, 8}, clip in {1, 2, 4} std; then the entropy count, the parameter-server schemes
    and the 62-tensor layer-wise shape.  Kernel times are the library's own event pairs around each launch."""
    import torch
    from paper_1901_08924_b200 import lpc, synth
    res, roof = {}, []
    N = 8
    top = 28 if full else log2_len
    U = synth.gradient_vectors(N, 1 << top, "gauss", seed=1, device=dev)
    grid = {}

    def point(name, Uv, b, clip, reps=5):
        r = qa_point(dev, peak, Uv, b, clip, reps)
        grid[name] = r
        return r

    # the floor of a timed launch: the same calls on 8 x 2^10 values, where there is next to nothing to do
    r0 = qa_point(dev, peak, U[:, : 1 << 10], 4, 2.0, reps=20)
    res["launch_floor_us"] = {"workload": "N=8, len 2^10, b=4 (an event pair around a launch that has next to nothing to do)",
                              "quantize_fused_kernel (cooperative launch, one grid-wide hand-over)": round(r0["quantize_pack"]["one_launch_ms"] * 1e3, 2),
                              "unpack_average_prox_kernel (plain launch)": round(r0["unpack_average_prox"]["ms"] * 1e3, 2)}
    lens = [l for l in (16, 20, 24, 26, 28) if l <= top]
    for l2 in lens:
        r = point("gauss_len2^%d_b4_clip2" % l2, U[:, : 1 << l2], 4, 2.0, reps=10 if l2 <= 24 else 4)
        wl = "sweep N=8, len 2^%d, N(0,1), b=4, clip 2 std" % l2
        qp, ua = r["quantize_pack"], r["unpack_average_prox"]
        resident = r["l2_resident_input"]
        name = ("quantize_fused_kernel<4> (quantize+pack in one cooperative launch)" if qp["one_launch_ms"] > 0 else
                "quantize+pack (stats_kernel + finish_kernel + quantize_kernel<4>)")
        roof.append(roofline_entry(name, wl, qp["ms"] * 1e3, qp["bytes"], peak,
                                   note="input stays in L2 between the two looks at it: bound 4 + b/8 B per element; launch-bound at "
                                        "this size (see quantize_aggregate.launch_floor_us)" if resident else
                                   "two passes: 8 + b/8 B per element"))
        if not resident and qp["stats_ms"] > 0:
            roof.append(roofline_entry("stats_kernel", wl, qp["stats_ms"] * 1e3, N * (1 << l2) * 4, peak, "stats_kernel", N * (1 << l2)))
            roof.append(roofline_entry("quantize_kernel<4>", wl, qp["pack_ms"] * 1e3, N * (1 << l2) * 4.5, peak, "quantize_kernel<4>", N * (1 << l2)))
        roof.append(roofline_entry("unpack_average_prox_kernel<4>", wl, ua["ms"] * 1e3, ua["bytes"], peak,
                                   None if resident else "unpack_average_prox_kernel<4>", 1 << l2,
                                   note="launch-bound at this size" if resident else None))
    mid = min(26, top)
    Um = U[:, : 1 << mid]
    for b in (1, 2, 3, 8):
        r = point("gauss_len2^%d_b%d_clip2" % (mid, b), Um, b, 2.0)
        wl = "sweep N=8, len 2^%d, N(0,1), b=%d, clip 2 std" % (mid, b)
        roof.append(roofline_entry("quantize+pack, b=%d" % b, wl, r["quantize_pack"]["ms"] * 1e3, r["quantize_pack"]["bytes"], peak))
        if b == 3 and r["quantize_pack"]["pack_ms"] > 0:  # (a short vector goes through the one-launch path instead)
            roof.append(roofline_entry("quantize_kernel<3>", wl, r["quantize_pack"]["pack_ms"] * 1e3, N * (1 << mid) * (4 + 3 / 8), peak,
                                       "quantize_kernel<3>", N * (1 << mid)))
        roof.append(roofline_entry("unpack_average_prox_kernel<%d>" % b, wl, r["unpack_average_prox"]["ms"] * 1e3,
                                   r["unpack_average_prox"]["bytes"], peak, "unpack_average_prox_kernel<3>" if b == 3 else None, 1 << mid))
    if full:
        for clip in (1.0, 4.0):
            point("gauss_len2^%d_b4_clip%g" % (mid, clip), Um, 4, clip)
        del Um
        Ut = synth.gradient_vectors(N, 1 << mid, "student_t3", seed=2, device=dev)
        for clip in (1.0, 2.0, 4.0):
            point("student_t3_len2^%d_b4_clip%g" % (mid, clip), Ut, 4, clip)
        del Ut
    res["sweep_grid_N8"] = grid
    # ---- entropy count and the parameter-server schemes on 8 x 2^mid Gaussian vectors, b = 4, clip 2 std
    length, b = 1 << mid, 4
    Um = U[:, :length]
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.0, 0)
    _, stride = lpc.packed_layout(length, b)
    codes = torch.empty((N, stride), dtype=torch.int32, device=dev)
    delta = torch.empty((N, 1), dtype=torch.float32, device=dev)
    clipped = torch.empty((N, 1), dtype=torch.int32, device=dev)
    x = torch.zeros(length, device=dev)
    q.quantize_pack(Um, 1, codes_out=codes, delta_out=delta, clipped_out=clipped)
    hist = torch.empty((N, 1, 1 << b), dtype=torch.int64, device=dev)
    th = _kernel_ms(q, lambda i: q.message_entropy(codes, length, hist_out=hist, host_counts=False), 10, ("other",))["other"]
    _, ent, huf = q.message_entropy(codes, length, hist_out=hist)
    bh = N * length * b / 8
    res["entropy_count_N8_len2^%d_b4" % mid] = {
        "histogram": {"ms": round(th, 4), "bytes": bh, "gbs": round(bh / th * 1e-6, 1), "frac": round(bh / th * 1e-6 / peak, 4)},
        "bits_per_coordinate": {"raw": b, "entropy_bound": round(float(ent.mean()) / length, 4),
                                "huffman": round(float(huf.astype("float64").mean()) / length, 4)}}
    roof.append(roofline_entry("code_histogram_swar_kernel<4>", "8 x 2^%d 4-bit codes" % mid, th * 1e3, bh, peak,
                               "code_histogram_swar_kernel<4>", N * length))
    q.set_option(lpc.OPT_SHARED_SCALE, 1)
    tqs = _kernel_ms(q, lambda i: q.quantize_pack(Um, i, codes_out=codes, delta_out=delta, clipped_out=clipped), 4,
                     ("quant_stats", "other", "quant_pack", "quant_fused"))
    tqs = sum(tqs.values())
    bq = N * length * (8 + b / 8)
    ps = {"quantize_pack_unified_scale": {"ms": round(tqs, 4), "gbs": round(bq / tqs * 1e-6, 1), "frac": round(bq / tqs * 1e-6 / peak, 4)}}
    for name, scheme in (("scheme_b_sum", lpc.SCHEME_SERVER_SUM), ("scheme_c_requantize", lpc.SCHEME_SERVER_REQUANTIZE)):
        srv, bo = q.server_reduce(codes, length, scheme, 1)
        ts = _kernel_ms(q, lambda i: q.server_reduce(codes, length, scheme, 1, codes_out=srv), 10, ("aggregate",))["aggregate"]
        w = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 1, 1, bo, lpc.CLIP_NONE, 1.0, 0)
        if scheme == lpc.SCHEME_SERVER_SUM:
            w.set_option(lpc.OPT_AVERAGE_DIVISOR, N)
        d1 = delta[:1].contiguous()
        x2 = [x, torch.zeros(length, device=dev)]  # two iterates in turn: none finds its own last output in L2
        tw = _kernel_ms(w, lambda i: w.unpack_average_prox(srv, d1, length, x2[i % 2], 1.0, 1e-3), 10, ("aggregate",))["aggregate"]
        w.close()
        bs, bw = length * (N * b / 8 + bo / 8), length * (bo / 8 + 12)
        ps[name] = {"bits_back": bo,
                    "server": {"ms": round(ts, 4), "bytes": bs, "gbs": round(bs / ts * 1e-6, 1), "frac": round(bs / ts * 1e-6 / peak, 4)},
                    "worker_decode_prox": {"ms": round(tw, 4), "bytes": bw, "gbs": round(bw / tw * 1e-6, 1),
                                           "frac": round(bw / tw * 1e-6 / peak, 4)}}
        roof.append(roofline_entry("server_reduce4_kernel (%s)" % name, "8 x 2^%d 4-bit codes in, %d-bit stream out" % (mid, bo),
                                   ts * 1e3, bs, peak, "server_reduce4_kernel<7, sum>" if scheme == lpc.SCHEME_SERVER_SUM else None, length))
        del x2
    q.sync_status()
    res["parameter_server_N8_len2^%d_b4" % mid] = ps
    q.close()
    del U, Um, codes, x
    torch.cuda.empty_cache()
    if not full:
        res["roofline_kernels"] = roof
        return res
    # ---- layer-wise DNN-shaped aggregation: 62 tensors, 11.7M parameters, 16 workers, b = 4, clip 2.5 std per tensor
    N, b = 16, 4
    cur, snap, mu, offs = synth.dnn_gradients(N, seed=2, device=dev)
    total = offs[-1]
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.5, 0)
    _, stride = lpc.packed_layout(total, b, offs)
    codes = [torch.empty((N, stride), dtype=torch.int32, device=dev) for _ in range(2)]
    delta = torch.empty((N, len(offs) - 1), dtype=torch.float32, device=dev)
    clipped = torch.empty((N, len(offs) - 1), dtype=torch.int32, device=dev)
    xs = [torch.zeros(total, device=dev) for _ in range(4)]
    tq = _kernel_ms(q, lambda i: q.quantize_pack(cur, i, U_sub=snap, seg_offsets=offs, codes_out=codes[i % 2], delta_out=delta,
                                                 clipped_out=clipped), 10, ("quant_stats", "other", "quant_pack", "quant_fused"))
    tq = sum(tq.values())
    codes[1].copy_(codes[0])
    ta = _kernel_ms(q, lambda i: q.unpack_average_prox(codes[i % 2], delta, total, xs[i % 4], 0.1, 0.0, mu=mu, seg_offsets=offs), 20,
                    ("aggregate",))["aggregate"]
    q.sync_status()
    bq, ba = N * total * (16 + b / 8), total * (N * b / 8 + 16)  # aggregate: codes + mu + x read + x write
    res["dnn_62_tensors_N16_b4"] = {
        "quantize_pack": {"ms": round(tq, 4), "bytes": bq, "gbs": round(bq / tq * 1e-6, 1), "frac": round(bq / tq * 1e-6 / peak, 4),
                          "note": "u = cur - snap formed on the fly: 2 x 8 B read + b/8 B written per element"},
        "unpack_average_prox": {"ms": round(ta, 4), "bytes": ba, "gbs": round(ba / ta * 1e-6, 1), "frac": round(ba / ta * 1e-6 / peak, 4)},
        "combined_gbs": round((bq + ba) / (tq + ta) * 1e-6, 1)}
    wl = "62 tensors of an 18-layer residual network, 11.7M parameters, N=16, b=4, clip 2.5 std per tensor"
    roof.append(roofline_entry("quantize+pack with u = cur - snap (3 launches)", wl, tq * 1e3, bq, peak))
    roof.append(roofline_entry("unpack_average_prox_kernel<4> (+ mu)", wl, ta * 1e3, ba, peak))
    q.close()
    res["roofline_kernels"] = roof
    return res


def kernel_pass(dev, log2_len):
    """Every stand-alone kernel of the library twice, on 8 x 2^log2_len Gaussian values, in a fixed order and with no
    warm-up: the command that profiler captures of these kernels run (a few launches, a few hundred MB)."""
    import torch
    from paper_1901_08924_b200 import lpc, synth
    N, length = 8, 1 << log2_len
    U = synth.gradient_vectors(N, length, "gauss", seed=1, device=dev)
    x = torch.zeros(length, device=dev)
    done = []
    for b in (4, 3):
        q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.0, 0)
        for k in range(2):
            codes, delta, _ = q.quantize_pack(U, k)                 # stats_kernel, finish_kernel, quantize_kernel<b>
            q.unpack_average_prox(codes, delta, length, x, 1.0, 1e-3)  # unpack_average_prox_kernel<b>
        if b == 4:
            for k in range(2):
                q.message_entropy(codes, length, host_counts=False)  # code_histogram_swar_kernel<4>
            q.set_option(lpc.OPT_SHARED_SCALE, 1)
            codes, delta, _ = q.quantize_pack(U, 2)                  # + share_scale_kernel
            for k in range(2):
                q.server_reduce(codes, length, lpc.SCHEME_SERVER_SUM, k)         # server_reduce4_kernel<7, false>
                q.server_reduce(codes, length, lpc.SCHEME_SERVER_REQUANTIZE, k)  # server_reduce4_kernel<4, true>
        q.sync_status()
        q.close()
        done.append(b)
    short = min(length, 1 << 20)
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, 4, lpc.CLIP_STD, 2.0, 0)
    for k in range(2):
        q.quantize_pack(U[:, :short], k)                             # quantize_fused_kernel<4> (one cooperative launch)
    q.sync_status()
    one = q.query(lpc.INFO_QUANT_ONE_LAUNCH)
    q.close()
    return {"kernel_pass": "8 x 2^%d" % log2_len, "widths": done, "one_launch_on_2^20": one}


def tiny_logistic_bench(dev):
    """The small logistic workload (4,000 x 1,000, N = 4, B = 1, b = 2, clip 2.5 std, eta = 0.1): one epoch of m = 1,000
    inner steps after the snapshot pass, value only."""
    import torch
    from paper_1901_08924_b200 import lpc
    w = WORKLOADS["lpc_svrg_logistic_4000x1000_N4_B1_b2"]
    X, y, m, eta = make_problem(w, seed=0, device=dev)
    ctx = lpc.Context(X, y, loss_code(w), w["lam"], w["N"], w["B"], w["b"], lpc.CLIP_STD, w["c"], 0)
    st = torch.cuda.current_stream(dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    p0 = ctx.objective()
    for s in range(3):
        ctx.snapshot_full_grad()
        ctx.inner_steps(eta, s * m, m)
    ctx.sync_status()
    ev[0].record(st)
    for s in range(3, 8):
        ctx.snapshot_full_grad()
        ctx.inner_steps(eta, s * m, m)
    ev[1].record(st)
    ctx.sync_status()
    ms = ev[0].elapsed_time(ev[1]) / 5
    out = {"workload": "lpc_svrg_logistic_4000x1000_N4_B1_b2", "iters_per_s": round(m / (ms * 1e-3), 1), "epoch_ms": round(ms, 4),
           "step_us": round(ms * 1e3 / m, 3), "objective_start": p0, "objective_after_8_epochs": ctx.objective(),
           "loop_cluster_size": ctx.query(lpc.INFO_LOOP_CLUSTER_SIZE),
           "loop_coords_per_thread": ctx.query(lpc.INFO_LOOP_COORDS_PER_THREAD)}
    ctx.close()
    return out


def fused_large_batch_bench(dev, peak, n=65536, steps=30):
    """The fused worker kernel (sampling, SVRG difference, scale, quantize, pack) where it is bandwidth-bound: the ALPC
    workload's shape (d = 8,192, N = 32, logistic) with the minibatch raised to B = 256 rows per worker, so that one
    step gathers N*B*d*4 = 268 MB of rows, and to the kernel's limit of B = 1,024 (1.07 GB per step), where the
    fixed cost of a launch (sampling, first fills, scale exchange, packing) weighs less.  Times come from the
    library's per-kernel event profile."""
    import torch
    from paper_1901_08924_b200 import lpc, synth
    d, N = 8192, 32
    X, y, _ = synth.linear_problem(n, d, loss="logistic", sparsity=0.02, noise=0.1, seed=1, col_scale_range=(0.1, 10.0),
                                   device=dev)
    out = {"workload": "fused_step_logistic_%dx8192_N32" % n, "roofline_kernels": []}
    for B, bits in ((256, (2, 8)), (1024, (2,))):
        if N * B > n:  # a small matrix for profiler captures: the larger minibatch does not fit its row partitions
            continue
        for b in bits:
            ctx = lpc.Context(X, y, lpc.LOGISTIC, 1e-5, N, B, b, lpc.CLIP_STD, 2.0, 0)
            ctx.snapshot_full_grad()
            ctx.inner_steps(1e-3, 0, 5)
            ctx.set_option(lpc.OPT_PROFILE, 1)
            ctx.inner_steps(1e-3, 5, steps)
            ctx.sync_status()
            prof = ctx.get_profile()
            tw = prof["worker"][0] / prof["worker"][1]
            ta = prof["aggregate"][0] / prof["aggregate"][1]
            bw = N * B * d * 4 + N * B * 8 + N * (d * b // 8 + 4)
            out["B%d_b%d" % (B, b)] = {"row_bytes_per_step": N * B * d * 4, "worker_us": round(tw * 1e3, 2),
                                       "worker_gbs": round(bw / tw * 1e-6, 1), "worker_frac": round(bw / tw * 1e-6 / peak, 4),
                                       "aggregate_us": round(ta * 1e3, 2), "ring_stages": ctx.query(lpc.INFO_STEP_RING_STAGES),
                                       "cluster_size": ctx.query(lpc.INFO_STEP_CLUSTER_SIZE)}
            out["roofline_kernels"].append(roofline_entry(
                "inner_kernel<%d, stream> (fused sampling + SVRG difference + scale + quantize + pack)" % b,
                "logistic %d x 8192, N=32 workers, B=%d rows per worker, b=%d" % (n, B, b), tw * 1e3, bw, peak,
                "inner_kernel<2, stream>" if b == 2 else None, N * B))
            ctx.close()
    return out


def alpc_bench(dev, peak):
    """ALPC-SVRG (Algorithms 2/3) on the ill-conditioned logistic workload: 262,144 x 8,192, N = 32, B = 16,
    clip 2 std, b in {2, 8}; one epoch = snapshot pass + m = n/(B N) = 512 double-sampling steps."""
    import torch
    from paper_1901_08924_b200 import lpc, synth
    n, d, N, B = 262144, 8192, 32, 16
    X, y, _ = synth.linear_problem(n, d, loss="logistic", sparsity=0.02, noise=0.1, seed=1, col_scale_range=(0.1, 10.0),
                                   device=dev)
    L = 0.25 * float((X * X).sum(dim=1).max().item())
    m = n // (B * N)
    out = {"workload": "alpc_svrg_logistic_262144x8192_N32_B16", "m": m, "roofline_kernels": []}
    for b in (2, 8):
        ctx = lpc.Context(X, y, lpc.LOGISTIC, 1e-5, N, B, b, lpc.CLIP_STD, 2.0, 0)
        ctx.alpc_begin()
        st = torch.cuda.current_stream(dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        times = []
        for s in range(5):  # Algorithm 3: tau1 = 2/(s+4), alpha = 1/(6 L tau1), tau2 = 1/2
            tau1 = 2.0 / (s + 4)
            ev[0].record(st)
            ctx.snapshot_full_grad()
            ev[1].record(st)
            ctx.alpc_double_sample_steps(tau1, 0.5, 1.0 / (6.0 * L * tau1), 1.0 / (4.0 * L), s * m, m)
            ctx.alpc_end_epoch(m)
            ev[2].record(st)
            torch.cuda.synchronize(dev)
            times.append((ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])))
        ctx.sync_status()
        snap = statistics.median(t[0] for t in times[2:])
        loop = statistics.median(t[1] for t in times[2:])
        out["b%d" % b] = {"iters_per_s": round(m / ((snap + loop) * 1e-3), 1), "step_us": round(loop * 1e3 / m, 3),
                          "snapshot_ms": round(snap, 4), "snapshot_gbs": round(n * d * 4 / snap * 1e-6, 1),
                          "loop_cluster_size": ctx.query(lpc.INFO_ALPC_LOOP_CLUSTER_SIZE),
                          "loop_row_slots": ctx.query(lpc.INFO_ALPC_LOOP_ROW_SLOTS),
                          "loop_coords_per_thread": ctx.query(lpc.INFO_ALPC_LOOP_COORDS_PER_THREAD),
                          "one_launch_loops": ctx.query(lpc.INFO_LOOP_LAUNCHES), "objective": ctx.objective()}
        step_bytes = (N + 1) * B * d * 4 + (N + 1) * B * 8 + 2 * N * (d // 8) * (1 if b <= 4 else 2) * 8 + 2 * d * 8
        out["roofline_kernels"].append(roofline_entry(
            "persist_kernel<%d, alpc> (one launch = %d steps of Algorithm 2)" % (b, m), out["workload"] + ", b=%d" % b,
            loop * 1e3, m * step_bytes, peak, note="latency chain per step: rows of N+1 minibatches, tagged code words "
            "written and read, second-estimator words"))
        if b == 2:
            out["roofline_kernels"].append(roofline_entry("snapshot_kernel", out["workload"], snap * 1e3, n * d * 4 + 8 * n + 4 * d,
                                                          peak, "snapshot_kernel (logistic)", n * d))
        ctx.close()
    # the strongly convex case (Algorithm 2, elastic net with sigma = L/1000, Theorem 3's tau1 and alpha)
    b, sigma = 2, L / 1000.0
    tau1 = min(0.5, (m * sigma / (6.0 * L)) ** 0.5)
    ctx = lpc.Context(X, y, lpc.LOGISTIC, 1e-5, N, B, b, lpc.CLIP_STD, 2.0, 0)
    ctx.set_strong_convexity(sigma)
    ctx.alpc_begin()
    st = torch.cuda.current_stream(dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    times = []
    for s in range(3):
        ctx.snapshot_full_grad()
        ev[0].record(st)
        ctx.alpc_double_sample_steps(tau1, 0.5, 1.0 / (6.0 * L * tau1), 1.0 / (4.0 * L), s * m, m)
        ctx.alpc_end_epoch(m)
        ev[1].record(st)
        torch.cuda.synchronize(dev)
        times.append(ev[0].elapsed_time(ev[1]))
    ctx.sync_status()
    out["strongly_convex_b2"] = {"sigma_over_L": 1e-3, "tau1": round(tau1, 4), "step_us": round(min(times[1:]) * 1e3 / m, 3),
                                 "one_launch_loops": ctx.query(lpc.INFO_LOOP_LAUNCHES), "objective": ctx.objective()}
    ctx.close()
    return out


def e2e_bench(w, X, y, m, eta, dev):
    """The whole job of the workload (5 epochs) through the host-buffer entry point: X, y copied in, x copied out."""
    import torch
    from paper_1901_08924_b200 import lpc
    S = 5
    Xh = torch.empty(X.shape, dtype=torch.float32, pin_memory=True)
    yh = torch.empty(y.shape, dtype=torch.float32, pin_memory=True)
    Xh.copy_(X)
    yh.copy_(y)
    x0 = torch.zeros(w["d"], dtype=torch.float32).pin_memory()
    torch.cuda.synchronize(dev)
    best = None
    for rep in range(2):  # first call warms the context up
        t0 = time.perf_counter()
        xh, P, bits = lpc.svrg_run_host(Xh, yh, loss_code(w), w["lam"], w["N"], w["B"], w["b"], lpc.CLIP_STD, w["c"], 0, S, m,
                                        eta, x0)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    h2d = Xh.numel() * 4 + yh.numel() * 4 + w["d"] * 4
    return {"value": round(S * m / best, 1), "unit": UNIT, "h2d_bytes_per_step": h2d // S, "d2h_bytes_per_step": (w["d"] * 4 + 8) // S,
            "job": "%d epochs via lpc_svrg_run_host from pinned host buffers, wall clock incl. allocation and copies" % S,
            "seconds": round(best, 4), "objective": P}


def oracle_epoch_sample(w, Xh, yh, m, eta, rows, steps, seed=0):
    """Times the oracle on a slice of one epoch: the full-gradient pass over `rows` rows and `steps` inner steps."""
    import numpy as np
    import oracle as orc
    code = orc.LEAST_SQUARES if w["loss"] == "least_squares" else orc.LOGISTIC
    P = orc.Problem(Xh, yh, code, w["lam"], w["N"], w["B"], w["b"], orc.CLIP_STD, w["c"], seed)
    x = np.zeros(w["d"], np.float32)
    t0 = time.perf_counter()
    mu, _, _ = orc.full_grad(Xh[:rows], yh[:rows], code, x)
    t_snap = time.perf_counter() - t0
    t0 = time.perf_counter()
    xs = x.copy()
    for k in range(steps):
        x = orc.lpc_inner_step(P, k, eta, x, xs, mu)
    t_inner = time.perf_counter() - t0
    return t_snap, t_inner


def cpu_baseline(w, X, y, m, eta):
    Xh, yh = X.cpu().numpy(), y.cpu().numpy()
    rows, steps = w["n"], m  # one whole epoch: about 10 s of single-core work on the main workload
    t_snap, t_inner = oracle_epoch_sample(w, Xh, yh, m, eta, rows, steps)
    epoch_s = t_snap * (w["n"] / rows) + t_inner * (m / steps)
    return {"value": round(m / epoch_s, 2), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "full-gradient pass over %d of %d rows (%.1f s) and %d of %d inner steps (%.1f s), scaled to one epoch"
                      % (rows, w["n"], t_snap, steps, m, t_inner)}


def run_reference(args):
    """The CPU oracle, as it stands, on the same workload and metric (rank 0 only)."""
    import torch
    from paper_1901_08924_b200 import dist_util
    size, rank, _ = dist_util.world()
    if rank != 0:
        return
    w = WORKLOADS[args.workload]
    X, y, m, eta = make_problem(w, seed=0, device="cpu")
    Xh, yh = X.numpy(), y.numpy()
    rows, steps = w["n"] // 32, max(1, m // 32)  # one step = 1/32 of an epoch
    times = []
    for i in range(max(args.warmup, 0) + args.steps):
        t_snap, t_inner = oracle_epoch_sample(w, Xh, yh, m, eta, rows, steps, seed=i)
        times.append(t_snap + t_inner)
    times = times[max(args.warmup, 0):]
    total = sum(times)
    value = args.steps * steps / total
    sample = "per step: full-gradient pass over %d of %d rows and %d of %d inner steps (1/32 epoch)" % (rows, w["n"], steps, m)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": size, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(total / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "n": w["n"], "d": w["d"], "N": w["N"], "B": w["B"], "b": w["b"]},
        "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--quick", action="store_true", help="skip the e2e, CPU-baseline and stand-alone kernel legs")
    ap.add_argument("--quantize-aggregate-only", type=int, default=0, metavar="LOG2LEN",
                    help="run only the stand-alone quantize+aggregate sweep point with 8 x 2^LOG2LEN values "
                         "(a small case for profiler captures)")
    ap.add_argument("--per-step-kernels", action="store_true",
                    help="run the inner loop as per-step kernels (graph replay) instead of the one-launch loop; "
                         "for profiler captures, which cannot replay the cooperative launch")
    ap.add_argument("--loop-not-cooperative", action="store_true",
                    help="launch the one-launch loop without the cooperative attribute (same grid, same kernel): for profiler "
                         "captures of it on a GPU that runs nothing else")
    ap.add_argument("--kernel-pass", type=int, default=0, metavar="LOG2LEN",
                    help="launch every stand-alone kernel twice on 8 x 2^LOG2LEN values (for profiler captures)")
    ap.add_argument("--alpc-only", action="store_true", help="run only the ALPC-SVRG leg (262,144 x 8,192)")
    ap.add_argument("--fused-large-batch-only", type=int, default=0, metavar="ROWS",
                    help="run only the large-minibatch leg of the fused worker kernel on a ROWS x 8192 matrix "
                         "(a small case for profiler captures)")
    args = ap.parse_args()
    if args.kernel_pass:
        import torch
        print(json.dumps(kernel_pass(torch.device("cuda", 0), args.kernel_pass)))
    elif args.fused_large_batch_only:
        import torch
        peak, _ = read_peak()
        print(json.dumps(fused_large_batch_bench(torch.device("cuda", 0), peak, n=args.fused_large_batch_only, steps=4)))
    elif args.quantize_aggregate_only:
        import torch
        peak, _ = read_peak()
        print(json.dumps(quantize_aggregate_bench(torch.device("cuda", 0), peak, args.quantize_aggregate_only, full=False)))
    elif args.alpc_only:
        import torch
        peak, _ = read_peak()
        print(json.dumps(alpc_bench(torch.device("cuda", 0), peak)))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
