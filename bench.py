#!/usr/bin/env python
"""Decode-step benchmark of the fused dequantize + mat-vec library.

One "step" = every mat-vec of one Llama-shaped decode step (7 per layer + lm_head), batch 1 by
default, issued through the C ABI (`lw_matvec`) on one stream and replayed as a CUDA graph.
Reports HBM GB/s (algorithmic bytes: weight bytes + 4*batch*(cols+rows) per call, over the step
time), decode-step-equivalent tokens/s, the roofline fraction against the measured HBM peak, an
end-to-end number with host<->device copies inside the timed region, and the CPU oracle timed on
the host cores as a reference baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--batch B]
    python bench.py --impl reference      # times the CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_20706_b200 import synth  # noqa: E402

METRIC = "mat-vec HBM GB/s (% of B200 peak) and decode-step-equiv tok/s, batch 1"
NOMINAL_PEAK_GBS = 8000.0
FALLBACK_PEAK_GBS = 6650.0
FMT_ID = {"f16": 0, "q8_0": 1, "q4_0": 2, "q4_K": 3, "q6_K": 4, "q5_K": 5, "q2_K": 6, "q4_1": 7, "q5_0": 8, "q5_1": 9}
BYTES_PER_WEIGHT = {"f16": 2.0, "q8_0": 34 / 32, "q4_0": 18 / 32, "q4_K": 144 / 256, "q6_K": 210 / 256, "q5_K": 176 / 256, "q2_K": 84 / 256, "q4_1": 20 / 32, "q5_0": 22 / 32, "q5_1": 24 / 32}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_PEAK_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def workload_spec(name, layers=None):
    factory, fmt, std, outlier_p, seed = synth.WORKLOADS[name]
    shapes = factory(layers) if layers else factory()
    return shapes, fmt, std, outlier_p, seed


def filter_shapes(shapes, only):
    if not only:
        return shapes
    keep = [s for s in shapes if any(tok in s[0] for tok in only.split(","))]
    if not keep:
        raise SystemExit("--only %r matches no mat-vec of the step" % only)
    return keep


def step_bytes(shapes, fmt, batch):
    """Algorithmic bytes of one step: every weight byte once + activations in/out once per call."""
    w = sum(int(r * c * BYTES_PER_WEIGHT[fmt]) for _, r, c in shapes)
    a = sum(4 * batch * (r + c) for _, r, c in shapes)
    return w, a


# ----------------------------------------------------------------------------- clocks ---

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            tok = [t.strip() for t in line.split(",")]
            if len(tok) < 8:
                continue
            try:
                sm.append(float(tok[0]))
                mx = float(tok[1])
            except ValueError:
                continue
            for name, val in zip(names, tok[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------- weight set (host) ---

def quantize_tensor(fmt_id, quantize_fn, row_bytes_fn, seed, tensor_id, rows, cols, std, outlier_p, out, pool):
    """Generate tensor `tensor_id` chunk by chunk and quantise it into `out` (uint8 view)."""
    n = rows * cols
    chunk = synth.CHUNK
    nchunks = (n + chunk - 1) // chunk

    def job(c):
        lo, hi = c * chunk, min(n, (c + 1) * chunk)
        x = synth.normal(seed, tensor_id, hi - lo, std, outlier_p, start=lo, threads=1)
        b0, b1 = row_bytes_fn(fmt_id, lo) if lo else 0, row_bytes_fn(fmt_id, hi)
        quantize_fn(fmt_id, x, out[b0:b1])

    list(pool.map(job, range(nchunks)))


# -------------------------------------------------------------------------- our arm ---

def run_ours(args):
    import torch

    from paper_2605_20706_b200 import lw

    from paper_2605_20706_b200 import dist_util
    rank, local_rank, world = dist_util.rank_info()
    if args.gpus != world and world > 1:
        log("warning: --gpus %d but WORLD_SIZE %d" % (args.gpus, world))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist_util.init("nccl", torch.device("cuda", local_rank))
    lw.lib()     # fail loudly here if the extension is missing

    shapes, fmt, std, outlier_p, seed = workload_spec(args.workload, args.layers)
    shapes = filter_shapes(shapes, args.only)
    fmt_id = FMT_ID[fmt]
    batch = args.batch
    ncalls = len(shapes)
    wbytes, abytes = step_bytes(shapes, fmt, batch)

    # ---- build the weight set: every matrix has its own memory (no aliasing between layers)
    t0 = time.time()
    offs, total = [], 0
    for _, r, c in shapes:
        offs.append(total)
        total += (lw.row_bytes(fmt_id, c) * r + 255) & ~255
    W = torch.empty(total, dtype=torch.uint8, device="cuda")
    max_mat = max(lw.row_bytes(fmt_id, c) * r for _, r, c in shapes)
    staging = torch.empty(max_mat, dtype=torch.uint8).pin_memory()
    stage_np = staging.numpy()
    keep_host = {}           # host copies of the first matrices, for the cpu_baseline / parity leg
    keep_budget = 600 << 20
    pool = ThreadPoolExecutor(max_workers=os.cpu_count() or 1)
    for i, (name, r, c) in enumerate(shapes):
        nb = lw.row_bytes(fmt_id, c) * r
        quantize_tensor(fmt_id, lw.quantize, lw.row_bytes, seed, i, r, c, std, outlier_p, stage_np[:nb], pool)
        W[offs[i]:offs[i] + nb].copy_(staging[:nb], non_blocking=True)
        if rank == 0 and keep_budget >= nb and (i < 7 or i == ncalls - 1):
            keep_host[i] = stage_np[:nb].copy()
            keep_budget -= nb
        torch.cuda.synchronize()
    pool.shutdown()
    log("weights: %d matrices, %.3f GB, built in %.1f s" % (ncalls, wbytes / 1e9, time.time() - t0))

    # ---- activations: one pinned host block with every call's X, one with every call's Y
    xoffs, yoffs, xt, yt = [], [], 0, 0
    for _, r, c in shapes:
        xoffs.append(xt)
        yoffs.append(yt)
        xt += (batch * c + 63) & ~63
        yt += (batch * r + 63) & ~63
    X_host = torch.empty(xt, dtype=torch.float32).pin_memory()
    Y_host = torch.empty(yt, dtype=torch.float32).pin_memory()
    xh = X_host.numpy()
    for i, (_, r, c) in enumerate(shapes):
        xh[xoffs[i]:xoffs[i] + batch * c] = synth.activations(seed, i, batch, c).reshape(-1)
    # q/k/v of a layer read the same activations, and so do gate/up: give them identical values
    for i in range(1, ncalls):
        leaf, prev = shapes[i][0].split(".")[-1], shapes[i - 1][0].split(".")[-1]
        if (leaf, prev) in (("k", "q"), ("v", "k"), ("up", "gate")) and shapes[i][2] == shapes[i - 1][2]:
            c = shapes[i][2]
            xh[xoffs[i]:xoffs[i] + batch * c] = xh[xoffs[i - 1]:xoffs[i - 1] + batch * c]
    X = X_host.cuda()
    Y = torch.zeros(yt, dtype=torch.float32, device="cuda")

    lw.set_overlap(not args.no_overlap)
    wptr, xptr, yptr = W.data_ptr(), X.data_ptr(), Y.data_ptr()

    # Mat-vecs that are independent in the model (q/k/v share one input, so do gate/up) are issued
    # on parallel branches; everything else stays in model order on the main branch.
    branch_of = []
    for name, _, _ in shapes:
        leaf = name.split(".")[-1]
        branch_of.append({"k": 1, "v": 2, "up": 1}.get(leaf, 0) if not args.serial else 0)
    aux = [torch.cuda.Stream(), torch.cuda.Stream()]

    def enqueue_per_call(stream):
        forked = set()
        for i, (_, r, c) in enumerate(shapes):
            b = branch_of[i]
            if b == 0:
                if forked:                      # join before the next dependent mat-vec
                    for j in sorted(forked):
                        ev = torch.cuda.Event()
                        ev.record(aux[j - 1])
                        stream.wait_event(ev)
                    forked.clear()
                target = stream
                # a following run of branch mat-vecs forks from the state before this launch
                if i + 1 < len(shapes) and branch_of[i + 1] != 0:
                    ev = torch.cuda.Event()
                    ev.record(stream)
                    j = i + 1
                    while j < len(shapes) and branch_of[j] != 0:
                        aux[branch_of[j] - 1].wait_event(ev)
                        j += 1
            else:
                target = aux[b - 1]
                forked.add(b)
            lw.matvec(fmt_id, wptr + offs[i], r, c, xptr + 4 * xoffs[i], yptr + 4 * yoffs[i], batch, target)
        for j in sorted(forked):
            ev = torch.cuda.Event()
            ev.record(aux[j - 1])
            stream.wait_event(ev)

    # Grouped issue: the same independent mat-vecs (q/k/v, gate/up) go into one lw_matvec_group call
    # each, everything else is a plain lw_matvec; one branch, model order.
    groups, i = [], 0
    while i < len(shapes):
        leaf = shapes[i][0].split(".")[-1]
        want = {"q": ["q", "k", "v"], "gate": ["gate", "up"]}.get(leaf)
        if want and [s[0].split(".")[-1] for s in shapes[i:i + len(want)]] == want \
                and len({s[2] for s in shapes[i:i + len(want)]}) == 1:
            groups.append(list(range(i, i + len(want))))
            i += len(want)
        else:
            groups.append([i])
            i += 1

    def enqueue_grouped(stream):
        for g in groups:
            if len(g) == 1:
                j = g[0]
                _, r, c = shapes[j]
                lw.matvec(fmt_id, wptr + offs[j], r, c, xptr + 4 * xoffs[j], yptr + 4 * yoffs[j], batch, stream)
            else:
                lw.matvec_group(fmt_id, shapes[g[0]][2],
                                [(wptr + offs[j], shapes[j][1], xptr + 4 * xoffs[j], yptr + 4 * yoffs[j]) for j in g],
                                stream)

    # Sequence issue: the whole chain in ONE lw_matvec_sequence call (persistent kernel); q/k/v and
    # gate/up share their X; every other mat-vec is flagged dependent on what came before it.
    seq_list = []
    for g in groups:
        for n, j in enumerate(g):
            _, r, c = shapes[j]
            x_of = g[0]          # the members of a group read the same activations
            seq_list.append((wptr + offs[j], r, c, xptr + 4 * xoffs[x_of], yptr + 4 * yoffs[j],
                             lw.SEQ_DEPENDENT if n == 0 else 0))
    seq_arr = lw.seq_items(seq_list)
    seq_ws = torch.zeros(lw.matvec_sequence_workspace_bytes() // 4, dtype=torch.int32, device="cuda")

    def enqueue_sequence(stream):
        lw.matvec_sequence(fmt_id, seq_arr, seq_ws, stream=stream)

    sequence = batch == 1 and args.issue == "sequence"
    grouped = batch == 1 and args.issue == "grouped"
    enqueue_step = enqueue_sequence if sequence else (enqueue_grouped if grouped else enqueue_per_call)
    launches_per_step = 1 if sequence else (len(groups) if grouped else ncalls)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        enqueue_step(side)
    side.synchronize()
    if lw.device_status() != 0:
        raise RuntimeError("device fault recorded during warm-up")
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            enqueue_step(side)

    stream = torch.cuda.current_stream()

    def one_step():
        if graph is not None:
            graph.replay()
        else:
            enqueue_step(stream)

    def barrier():
        torch.cuda.synchronize()
        dist_util.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    for _ in range(max(3, args.warmup)):
        one_step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        one_step()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    # keep the GPU busy a little longer so the clock sampler sees the loaded state
    t_end = time.time() + 1.0
    while time.time() < t_end:
        one_step()
    torch.cuda.synchronize()
    clocks = sampler.stop()

    # ---- the other issue mode (one call per mat-vec on parallel branches), for comparison
    other = None
    if grouped and graph is not None and not args.only:
        with torch.cuda.stream(side):
            enqueue_per_call(side)
        side.synchronize()
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=side):
            enqueue_per_call(side)
        for _ in range(3):
            g2.replay()
        barrier()
        o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        o0.record(stream)
        for _ in range(args.steps):
            g2.replay()
        o1.record(stream)
        barrier()
        oms = o0.elapsed_time(o1) / args.steps
        other = {"issue": "one lw_matvec call per mat-vec (%d launches per step), q/k/v and gate/up on parallel "
                          "graph branches" % ncalls,
                 "ms_per_step": round(oms, 5), "value": round((wbytes + abytes) / (oms * 1e-3) / 1e9, 1),
                 "unit": "GB/s", "tok_per_s": round(1e3 / oms, 2)}

    # ---- end to end: host activations in, host results out, every step
    for _ in range(3):
        X.copy_(X_host, non_blocking=True)
        one_step()
        Y_host.copy_(Y, non_blocking=True)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        X.copy_(X_host, non_blocking=True)
        one_step()
        Y_host.copy_(Y, non_blocking=True)
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    if lw.device_status() != 0:
        raise RuntimeError("device fault recorded during the timed region")

    ms, ms_e2e = dist_util.max_over_ranks([ms, ms_e2e], device="cuda")

    step_ms = ms / args.steps
    total_bytes = (wbytes + abytes) * world
    gbs = total_bytes / (step_ms * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    per_gpu_gbs = gbs / world
    result = {
        "metric": METRIC,
        "value": round(gbs, 1),
        "unit": "GB/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": max(3, args.warmup),
        "ms_per_step": round(step_ms, 5),
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "f32",
        "data": "synthetic",
        "config": {
            "workload": "%s: %d mat-vecs per decode step, batch %d, weights %.3f GB in %s, "
                        "fp32 activations; %s%s%s" % (
                            args.workload, ncalls, batch, wbytes / 1e9, fmt,
                            ("lw_matvec_group for q/k/v and for gate/up (independent in the model), lw_matvec for "
                             "the rest: %d launches per step" % launches_per_step) if grouped
                            else "one lw_matvec call per mat-vec",
                            ", replayed as one CUDA graph" if graph is not None else "",
                            (", programmatic dependent launch between calls" if not args.no_overlap else "") +
                            ("" if (args.serial or grouped) else "; q/k/v and gate/up (independent in the model) on parallel graph branches")),
            "format": fmt, "batch": batch, "calls_per_step": ncalls,
            "weight_bytes": wbytes, "activation_bytes": abytes,
            "l2": "weight set is %.0fx the 126 MB L2 and is streamed evict-first; no flush needed" % (wbytes / 126e6),
            "parallelism": "replicas only (one independent decode step per GPU)" if world > 1 else "single GPU",
        },
        "tok_per_s": round(world * 1e3 / step_ms, 2),
        "pct_of_nominal_8TBs": round(100 * per_gpu_gbs / NOMINAL_PEAK_GBS, 2),
        "effective_gflops": round(world * sum(2.0 * r * c * batch for _, r, c in shapes) / (step_ms * 1e-3) / 1e9, 1),
        "clocks": clocks,
        "gpu_launches": args.steps * launches_per_step,
        "per_call": other,
        "e2e": {
            "value": round((wbytes + abytes) * world / (ms_e2e / args.steps * 1e-3) / 1e9, 1),
            "unit": "GB/s",
            "ms_per_step": round(ms_e2e / args.steps, 5),
            "tok_per_s": round(world * args.steps * 1e3 / ms_e2e, 2),
            "h2d_bytes_per_step": int(X_host.numel() * 4),
            "d2h_bytes_per_step": int(Y_host.numel() * 4),
        },
        "roofline": {
            "bound": "hbm",
            "achieved": round(per_gpu_gbs, 1),
            "peak": peak,
            "peak_source": peak_src,
            "unit": "GB/s",
            "frac": round(per_gpu_gbs / peak, 4),
            "traffic": (int(TRAFFIC_RATIO[args.workload] * (wbytes + abytes) / launches_per_step)
                        if args.workload in TRAFFIC_RATIO and batch == 1 else None),
            "kernel": "matvec_stream_kernel<%s%s>" % ("Idot_" if fmt != "f16" and batch == 1 else "", fmt),
            "bytes_per_launch_avg": int((wbytes + abytes) / launches_per_step),
        },
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline_leg(shapes, fmt, fmt_id, batch, seed, std, outlier_p, keep_host, xh,
                                                  xoffs, Y, yoffs, args.cpu_seconds)
    if rank == 0:
        print(json.dumps(result), flush=True)
    dist_util.shutdown()


# Measured DRAM bytes (read + write) per algorithmic byte of the dominant kernel, from the ncu capture
# summarised under profiles/ (taken on two matrices of the workload and scaled by bytes, since DRAM
# traffic of this streaming kernel grows in proportion to the bytes it processes).
TRAFFIC_RATIO = {"llama8b_q4_K": 1.010}


# --------------------------------------------------------- oracle legs (CPU, rank 0) ---

def cpu_baseline_leg(shapes, fmt, fmt_id, batch, seed, std, outlier_p, keep_host, xh, xoffs, Y_dev, yoffs,
                     seconds):
    """Times the oracle (as it stands) on a bounded sample of the step -- whole matrices, regenerated
    from the seeded recipe and quantised by the oracle's own quantiser -- and checks the GPU results
    of those matrices against it with the mat-vec tolerance."""
    import oracle
    cores = os.cpu_count() or 1
    total_w = sum(r * c for _, r, c in shapes)
    pool = ThreadPoolExecutor(max_workers=cores)

    def oracle_quant(f, x, out):
        out[:] = oracle.quantize(f, x)

    def make(i):
        _, r, c = shapes[i]
        out = np.empty(oracle.row_bytes(fmt_id, c) * r, dtype=np.uint8)
        quantize_tensor(fmt_id, oracle_quant, oracle.row_bytes, seed, i, r, c, std, outlier_p, out, pool)
        return out

    order = list(range(min(7, len(shapes)))) + ([len(shapes) - 1] if len(shapes) > 7 else [])
    order += [i for i in range(7, len(shapes) - 1)]
    y_gpu = Y_dev.cpu().numpy()
    worst, cpu_time, nbytes, used, chosen, bytes_equal = 0.0, 0.0, 0, 0, [], True
    t_leg = time.time()
    for i in order:
        _, r, c = shapes[i]
        if chosen and cpu_time > 0 and cpu_time * (1 + r * c / max(used, 1)) > seconds:
            break
        if time.time() - t_leg > 4 * seconds:
            break
        blocks = make(i)
        if i in keep_host:
            bytes_equal = bytes_equal and bool((blocks == keep_host[i]).all())
        x = xh[xoffs[i]:xoffs[i] + batch * c]
        t = time.time()
        y_ref, s_ref = oracle.matvec(fmt_id, blocks, r, c, x, batch, nthreads=cores)
        cpu_time += time.time() - t
        nbytes += int(r * c * BYTES_PER_WEIGHT[fmt]) + 4 * batch * (r + c)
        used += r * c
        chosen.append(i)
        got = y_gpu[yoffs[i]:yoffs[i] + batch * r].reshape(batch, r).astype(np.float64)
        worst = max(worst, float((np.abs(got - y_ref) / (1e-4 * s_ref + 1e-6)).max()))
    pool.shutdown()
    return {
        "value": round(nbytes / cpu_time / 1e9, 4),
        "unit": "GB/s",
        "cores": cores,
        "kind": "oracle",
        "sample": "%d of the step's %d mat-vecs (first layer, lm_head, then further layers in order; "
                  "%.1f%% of the step's weights), every row; %.1f s of oracle mat-vec time" % (
                      len(chosen), len(shapes), 100.0 * used / total_w, cpu_time),
        "tok_per_s_equiv": round(1.0 / (cpu_time * total_w / used), 5),
        "gpu_vs_oracle_worst_err_over_tol": round(worst, 4),
        "parity_ok": bool(worst <= 1.0),
        "host_quantiser_bytes_equal_oracle": bytes_equal,
    }


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    shapes, fmt, std, outlier_p, seed = workload_spec(args.workload, args.layers)
    fmt_id = FMT_ID[fmt]
    batch = args.batch
    cores = os.cpu_count() or 1
    # sample: the first layer's matrices, rows capped so that one step takes a few seconds
    sample = [(i, shapes[i]) for i in range(min(7, len(shapes)))]
    mats = []
    for i, (name, r, c) in sample:
        rr = min(r, args.ref_rows)
        w = synth.normal(seed, i, rr * c, std, outlier_p).reshape(rr, c)     # first rr rows of the tensor
        x = synth.activations(seed, i, batch, c)
        mats.append((oracle.quantize(fmt_id, w), rr, c, x))
    nbytes = sum(int(rr * c * BYTES_PER_WEIGHT[fmt]) + 4 * batch * (rr + c) for _, rr, c, _ in mats)
    nweights = sum(rr * c for _, rr, c, _ in mats)

    def step():
        for blocks, rr, c, x in mats:
            oracle.matvec(fmt_id, blocks, rr, c, x, batch, nthreads=cores)

    for _ in range(max(1, args.warmup)):
        step()
    t = time.time()
    for _ in range(args.steps):
        step()
    dt = (time.time() - t) / args.steps
    gbs = nbytes / dt / 1e9
    total_w = sum(r * c for _, r, c in shapes)
    sample_txt = ("first %d rows of each of the first layer's 7 matrices (%d weights = %.3f%% of a step) per "
                  "step" % (args.ref_rows, nweights, 100.0 * nweights / total_w))
    print(json.dumps({
        "impl": "reference",
        "metric": METRIC, "value": round(gbs, 4), "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": max(1, args.warmup),
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s (CPU oracle on a bounded sample: %s)" % (args.workload, sample_txt),
                   "format": fmt, "batch": batch},
        "tok_per_s": round(nweights / total_w / dt, 5),
        "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)



# ------------------------------------------------------------- decode attention workloads ---

ATTN_METRIC = "decode-attention HBM GB/s over a block-quantised KV cache (% of B200 peak), one query token"


def attn_bytes(n_head, n_kv, hd, n_pos, fmt):
    """Algorithmic bytes of one call: both caches once, the query in, the output out."""
    cache = 2 * n_pos * int(n_kv * hd * BYTES_PER_WEIGHT[fmt])
    return cache, 8 * n_head * hd


def run_attn(args):
    """One "step" = one lw_attn_decode call per layer, each layer with its own K and V cache."""
    import torch

    from paper_2605_20706_b200 import dist_util, lw
    rank, local_rank, world = dist_util.rank_info()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist_util.init("nccl", torch.device("cuda", local_rank))
    lw.lib()
    n_head, n_kv, hd, n_pos, layers, fmt, seed = synth.ATTN_WORKLOADS[args.workload]
    if args.layers:
        layers = args.layers
    fmt_id = FMT_ID[fmt]
    width = n_kv * hd
    scale = 1.0 / float(np.sqrt(hd))
    cbytes, qbytes = attn_bytes(n_head, n_kv, hd, n_pos, fmt)
    t0 = time.time()
    Ks, Vs, host_kv = [], [], None
    for layer in range(layers):
        kb = lw.quantize(fmt_id, synth.kv_cache(seed, 2 * layer, n_pos, width))
        vb = lw.quantize(fmt_id, synth.kv_cache(seed, 2 * layer + 1, n_pos, width))
        Ks.append(torch.from_numpy(kb).cuda())
        Vs.append(torch.from_numpy(vb).cuda())
        if layer == 0:
            host_kv = (kb, vb)
    log("caches: %d layers x 2 x %.1f MB in %s, built in %.1f s" % (layers, cbytes / 2e6, fmt, time.time() - t0))
    Q_host = torch.empty(layers, n_head, hd, dtype=torch.float32).pin_memory()
    O_host = torch.empty(layers, n_head, hd, dtype=torch.float32).pin_memory()
    for layer in range(layers):
        Q_host[layer] = torch.from_numpy(synth.query(seed, layer, n_head, hd))
    Q = Q_host.cuda()
    O = torch.zeros(layers, n_head, hd, dtype=torch.float32, device="cuda")
    ws = torch.empty(lw.attn_workspace_bytes(n_head, n_kv, hd, n_pos) // 4, dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    variant = lw.query_attn_variant(fmt_id, n_head, n_kv, hd, n_pos)

    def enqueue(st):
        for layer in range(layers):
            lw.attn_decode(fmt_id, Ks[layer], Vs[layer], Q[layer], O[layer], n_head, n_kv, hd, n_pos, scale, ws, stream=st)

    def barrier():
        torch.cuda.synchronize()
        dist_util.barrier()

    with torch.cuda.stream(stream):
        enqueue(stream)
    barrier()
    # ---- parity of layer 0 against the oracle on the same buffers (rank 0, single GPU runs)
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        ref, S = oracle.attn_decode(fmt_id, host_kv[0], host_kv[1], Q_host[0].numpy(), n_head, n_kv, hd, n_pos, scale)
        got = O[0].double().cpu().numpy()
        parity = float((np.abs(got - ref) / (1e-4 * S + 1e-6)).max())
        if not parity <= 1.0:
            raise RuntimeError("parity check failed: worst error / tolerance = %.3g" % parity)
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            enqueue(torch.cuda.current_stream())

    def one_step():
        if graph is not None:
            graph.replay()
        else:
            enqueue(stream)

    with torch.cuda.stream(stream):
        for _ in range(max(3, args.warmup)):
            one_step()
        barrier()
        sampler = ClockSampler(local_rank)
        sampler.start()
        time.sleep(0.3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(args.steps):
            one_step()
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        t_busy = time.time() + 1.0             # keep the GPU busy a little longer so the sampler sees the loaded state
        while time.time() < t_busy:
            one_step()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        # ---- end to end: the queries come from pinned host memory and the outputs go back, every step
        for _ in range(3):
            Q.copy_(Q_host, non_blocking=True)
            one_step()
            O_host.copy_(O, non_blocking=True)
        barrier()
        e0.record(stream)
        for _ in range(args.steps):
            Q.copy_(Q_host, non_blocking=True)
            one_step()
            O_host.copy_(O, non_blocking=True)
        e1.record(stream)
        barrier()
        ms_e2e = e0.elapsed_time(e1)
    if lw.device_status() != 0:
        raise RuntimeError("device fault recorded during the timed region")
    ms, ms_e2e = dist_util.max_over_ranks([ms, ms_e2e], device="cuda")
    step_ms = ms / args.steps
    step_bytes_ = layers * (cbytes + qbytes)
    gbs = world * step_bytes_ / (step_ms * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    kernel = ("attn_decode_mma_kernel<%s, %d>" % (fmt, hd)) if variant == 2 else ("attn_decode_general_kernel<%s>" % fmt)
    result = {
        "metric": ATTN_METRIC, "value": round(gbs, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": round(step_ms, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": "%s: %d lw_attn_decode calls per step (one per layer, own K and V cache each), %d query heads "
                        "over %d KV heads of %d dims, %d cached positions in %s (%.1f MB per call)%s" % (
                            args.workload, layers, n_head, n_kv, hd, n_pos, fmt, cbytes / 1e6,
                            ", replayed as one CUDA graph" if graph is not None else ""),
            "format": fmt, "calls_per_step": layers, "cache_bytes_per_call": cbytes,
            "l2": "the step's caches are %.1fx the 126 MB L2; every call reads its own" % (layers * cbytes / 126e6),
            "parallelism": "replicas only (one independent step per GPU)" if world > 1 else "single GPU",
        },
        "us_per_call": round(1e3 * step_ms / layers, 2),
        "clocks": clocks,
        "gpu_launches": args.steps * layers * 2,
        "parity_worst_error_over_tolerance": None if parity is None else round(parity, 4),
        "e2e": {"value": round(world * step_bytes_ / (ms_e2e / args.steps * 1e-3) / 1e9, 1), "unit": "GB/s",
                "ms_per_step": round(ms_e2e / args.steps, 5), "h2d_bytes_per_step": int(Q_host.numel() * 4),
                "d2h_bytes_per_step": int(O_host.numel() * 4)},
        "roofline": {"bound": "hbm", "achieved": round(gbs / world, 1), "peak": peak, "peak_source": peak_src,
                     "unit": "GB/s", "frac": round(gbs / world / peak, 4),
                     "traffic": (int(ATTN_TRAFFIC_RATIO[args.workload] * (cbytes + qbytes))
                                 if args.workload in ATTN_TRAFFIC_RATIO else None),
                     "kernel": kernel, "bytes_per_launch_avg": int(cbytes + qbytes)},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = attn_cpu_leg(args.workload, args.cpu_seconds)
    if rank == 0:
        print(json.dumps(result), flush=True)
    dist_util.shutdown()


# DRAM bytes (read + write) per algorithmic byte of the attention kernel, from the ncu capture under profiles/.
ATTN_TRAFFIC_RATIO = {"attn8b_q8_0_ctx32k": 1.017}


def attn_sample(workload, positions):
    """Oracle-side sample of an attention workload: the first `positions` cached positions of layer 0."""
    import oracle
    n_head, n_kv, hd, n_pos, layers, fmt, seed = synth.ATTN_WORKLOADS[workload]
    fmt_id = FMT_ID[fmt]
    n = min(n_pos, positions)
    width = n_kv * hd
    K = oracle.quantize(fmt_id, synth.kv_cache(seed, 0, n, width))
    V = oracle.quantize(fmt_id, synth.kv_cache(seed, 1, n, width))
    q = synth.query(seed, 0, n_head, hd)
    cbytes, qbytes = attn_bytes(n_head, n_kv, hd, n, fmt)
    return (fmt_id, K, V, q, n_head, n_kv, hd, n, 1.0 / float(np.sqrt(hd))), cbytes + qbytes, n, n_pos * layers


def attn_cpu_leg(workload, seconds):
    """Times the oracle's attention (as it stands: numpy on the host cores) on a bounded sample."""
    import oracle
    call, nbytes, n, total = attn_sample(workload, 8192)
    oracle.attn_decode(*call)
    reps, t = 0, time.time()
    while reps < 1 or time.time() - t < seconds:
        oracle.attn_decode(*call)
        reps += 1
    dt = (time.time() - t) / reps
    return {"value": round(nbytes / dt / 1e9, 4), "unit": "GB/s", "cores": os.cpu_count() or 1, "kind": "oracle",
            "sample": "layer 0, first %d cached positions (%.3f%% of a step's positions), %d repetitions" % (
                n, 100.0 * n / total, reps)}


def run_attn_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    call, nbytes, n, total = attn_sample(args.workload, 8192)
    for _ in range(max(1, args.warmup)):
        oracle.attn_decode(*call)
    t = time.time()
    for _ in range(args.steps):
        oracle.attn_decode(*call)
    dt = (time.time() - t) / args.steps
    gbs = nbytes / dt / 1e9
    sample_txt = "layer 0, first %d cached positions (%.3f%% of a step's positions) per step" % (n, 100.0 * n / total)
    print(json.dumps({
        "impl": "reference", "metric": ATTN_METRIC, "value": round(gbs, 4), "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": max(1, args.warmup),
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s (CPU oracle on a bounded sample: %s)" % (args.workload, sample_txt)},
        "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "cores": os.cpu_count() or 1, "kind": "oracle",
                         "sample": sample_txt},
        "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_q4_K",
                    choices=sorted(synth.WORKLOADS) + sorted(synth.ATTN_WORKLOADS))
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=None, help="use fewer layers (debugging only)")
    ap.add_argument("--only", default=None, help="comma-separated substrings: keep only matching mat-vecs "
                                                  "(profiling of single kernels)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--issue", default="sequence", choices=["sequence", "grouped", "per-call"],
                    help="sequence: one lw_matvec_sequence call per step; grouped: lw_matvec_group for q/k/v and "
                         "gate/up, lw_matvec for the rest; per-call: one lw_matvec per mat-vec")
    ap.add_argument("--serial", action="store_true", help="one branch: every mat-vec waits for the previous one")
    ap.add_argument("--no-overlap", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=4.0)
    ap.add_argument("--ref-rows", type=int, default=512)
    args = ap.parse_args()
    attn = args.workload in synth.ATTN_WORKLOADS
    if args.impl == "reference":
        (run_attn_reference if attn else run_reference)(args)
    else:
        (run_attn if attn else run_ours)(args)


if __name__ == "__main__":
    main()
