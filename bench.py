#!/usr/bin/env python
"""Benchmarks of the fused dequantize + mat-vec library.

Default workload: the decode step.  One "step" = every mat-vec of one Llama-shaped decode step (7 per
layer + lm_head), batch 1 by default, issued through the C ABI on one stream and replayed as a CUDA
graph.  Reports HBM GB/s (algorithmic bytes: weight bytes + 4*batch*(cols+rows) per call, over the step
time), decode-step-equivalent tokens/s, the roofline fraction against the measured HBM peak (and the
read-only ceiling of the copy pipeline), an end-to-end number through the host-buffer C-ABI call with the
host<->device copies inside the timed region, and the CPU oracle timed on the host cores as a reference.

Issue modes of the step (batch 1): `launches` = one lw_matvec_sequence call per step, implemented as one
grouped launch per phase chained with programmatic dependent launch (LW_SEQ_LAUNCHES, the library's
default), `persistent` = the same call as one persistent kernel (LW_SEQ_PERSISTENT), `per-call` = one
lw_matvec per mat-vec.  `auto` (default) times launches and persistent and reports the faster one as the
headline.

Other workloads: `q8_0_2048` (one 2048x2048 q8_0 mat-vec: hot-L2 latency and a cold figure rotating over
64 copies), `dequant_<fmt>` (stand-alone dequantisation), `attn*` (decode attention).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--batch B] [--issue MODE]
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
SINGLE_WORKLOADS = ("q8_0_2048",)
DEQUANT_WORKLOADS = tuple("dequant_" + f for f in FMT_ID)


MMA_FORMATS = ("q8_0", "q4_0", "q4_K", "q5_K", "f16", "q4_1", "q5_0", "q5_1", "q6_K", "q2_K")       # formats the batched tensor-core kernel takes


def arithmetic_of(fmt, batch):
    """What the kernels compute in (the `dtype` key): not a precision claim, the arithmetic that runs."""
    if fmt == "f16" and batch >= 3:
        return ("f32 in/out; f16 weights x two-term f16 split of the block-scaled fp32 activations on the tensor cores "
                "(mma m16n8k16), fp32 accumulation")
    if fmt == "f16":
        return "f32 in/out; f16 weights widened, fp32 FMA"
    if batch == 1:
        return "f32 in/out; activations as 24-bit block fixed point, int32 dp4a sums, fp32 block scales"
    if fmt in MMA_FORMATS and batch >= 3:
        return ("f32 in/out; exact bf16 weight codes x two-term bf16 split (16 significant bits) of the fp32 activations on the tensor cores "
                "(mma m16n8k16), fp32 accumulation and block scales")
    return "f32 in/out; batch > 1: per-column passes of the batch-1 kernel (24-bit block fixed point, int32 dp4a) or fp32 FMA tiles"


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


# ----------------------------------------------------------------------- common pieces ---

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


def device_setup():
    import torch

    from paper_2605_20706_b200 import dist_util, lw
    rank, local_rank, world = dist_util.rank_info()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist_util.init("nccl", torch.device("cuda", local_rank))
    lw.lib()     # fail loudly here if the extension is missing
    return torch, dist_util, lw, rank, local_rank, world


class Timer:
    """CUDA-event timing of a callable on the current stream, warm-up first, barrier + synchronize on both sides."""

    def __init__(self, torch, dist_util):
        self.torch, self.dist = torch, dist_util
        self.stream = torch.cuda.current_stream()

    def barrier(self):
        self.torch.cuda.synchronize()
        self.dist.barrier()
        self.torch.cuda.synchronize()

    def time(self, fn, steps, warmup):
        for _ in range(max(3, warmup)):
            fn()
        self.barrier()
        e0, e1 = self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for _ in range(steps):
            fn()
        e1.record(self.stream)
        self.barrier()
        return e0.elapsed_time(e1) / steps       # ms per call of fn


def capture(torch, enqueue, use_graph=True):
    """Runs `enqueue(stream)` once on a side stream (warm-up outside capture), then captures it into a graph;
    returns a callable that replays it on the current stream."""
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        enqueue(side)
    side.synchronize()
    if not use_graph:
        cur = torch.cuda.current_stream()
        return lambda: enqueue(cur)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        enqueue(side)
    return graph.replay


def read_only_ceiling(lw, timer, buf, nbytes):
    """GB/s of the streaming kernels' copy pipeline with no arithmetic behind it, over `nbytes` of `buf`."""
    nbytes -= nbytes % 16
    if nbytes < (256 << 20):
        return None
    ms = timer.time(lambda: lw.probe_read(buf, nbytes), 5, 3)
    return round(nbytes / (ms * 1e-3) / 1e9, 1)


def roofline_block(per_gpu_gbs, kernel, bytes_per_launch, traffic, ceiling=None, bound="hbm"):
    peak, peak_src = measured_peak()
    out = {"bound": bound, "achieved": round(per_gpu_gbs, 1), "peak": peak, "peak_source": peak_src, "unit": "GB/s",
           "frac": round(per_gpu_gbs / peak, 4), "traffic": traffic, "kernel": kernel,
           "bytes_per_launch_avg": int(bytes_per_launch),
           "frac_of_nominal_8000": round(per_gpu_gbs / NOMINAL_PEAK_GBS, 4)}
    if ceiling:
        out["read_only_ceiling"] = {"value": ceiling, "unit": "GB/s", "frac_of_it": round(per_gpu_gbs / ceiling, 4),
                                    "what": "lw_probe_read over the workload's weights: the same bulk-copy rings, no arithmetic"}
    return out


# DRAM bytes (read + write) per algorithmic byte of the dominant kernel, from the ncu captures summarised under
# profiles/ (taken on a few matrices of the workload and scaled by bytes: DRAM traffic of these streaming
# kernels grows in proportion to the bytes they process).
TRAFFIC_RATIO = {"llama8b_q4_K": 1.010}


# ------------------------------------------------------------------ the decode step ---

def run_step(args):
    torch, dist_util, lw, rank, local_rank, world = device_setup()
    if args.gpus != world:
        log("note: --gpus %d, running with WORLD_SIZE %d" % (args.gpus, world))
    shapes, fmt, std, outlier_p, seed = workload_spec(args.workload, args.layers)
    shapes = filter_shapes(shapes, args.only)
    fmt_id = FMT_ID[fmt]
    batch = args.batch
    ncalls = len(shapes)
    wbytes, abytes = step_bytes(shapes, fmt, batch)
    timer = Timer(torch, dist_util)

    # ---- weights: every matrix has its own memory (no aliasing between layers)
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

    # batch > 1: the weights are model parameters that nothing on the stream writes, so the tensor-core kernel may
    # start streaming them while the previous kernel finishes (overlap level 2)
    overlap_level = 0 if args.no_overlap else (args.overlap if args.overlap is not None else (2 if batch > 1 else 1))
    lw.set_overlap(overlap_level)
    if args.tuning_table:
        log("tuning table: %d entries" % lw.load_tuning_table(args.tuning_table))
    wptr, xptr, yptr = W.data_ptr(), X.data_ptr(), Y.data_ptr()
    xhptr, yhptr = X_host.data_ptr(), Y_host.data_ptr()

    # Mat-vecs that are independent in the model (q/k/v share one input, so do gate/up) are issued on parallel
    # branches in per-call mode; everything else stays in model order on the main branch.
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

    # Groups: the independent mat-vecs that share their activations (q/k/v, gate/up); everything else alone.
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

    # Sequence: the whole chain in ONE lw_matvec_sequence call; the members of a group read one X, the first
    # member of every group is flagged dependent on everything before it.
    seq_list = []
    for g in groups:
        for n, j in enumerate(g):
            _, r, c = shapes[j]
            seq_list.append((wptr + offs[j], r, c, xptr + 4 * xoffs[g[0]], yptr + 4 * yoffs[j],
                             lw.SEQ_DEPENDENT if n == 0 else 0))
    seq_arr = lw.seq_items(seq_list)
    seq_ws = torch.zeros(lw.matvec_sequence_workspace_bytes() // 4, dtype=torch.int32, device="cuda")

    def enqueue_launches(stream):
        lw.set_sequence_mode(lw.SEQ_LAUNCHES)
        lw.matvec_sequence(fmt_id, seq_arr, seq_ws, stream=stream)

    def enqueue_persistent(stream):
        lw.set_sequence_mode(lw.SEQ_PERSISTENT)
        lw.matvec_sequence(fmt_id, seq_arr, seq_ws, stream=stream)

    def enqueue_grouped(stream):
        # batch > 1: ONE lw_matvec_sequence_batch call per step, which makes one lw_matvec_group_batch call per group
        # (q/k/v together, gate/up together, the rest alone)
        lw.matvec_sequence_batch(fmt_id, seq_arr, batch, stream)

    modes = {"launches": (enqueue_launches, len(groups),
                          "one lw_matvec_sequence call per step, run as one grouped launch per phase (q/k/v together, "
                          "gate/up together, the rest alone: %d launches per step) chained with programmatic dependent "
                          "launch" % len(groups)),
             "persistent": (enqueue_persistent, 1,
                            "one lw_matvec_sequence call per step, run as ONE persistent kernel (grid-wide barrier before "
                            "each dependent mat-vec, weight ring kept filling across boundaries): 1 launch per step"),
             "per-call": (enqueue_per_call, ncalls, "one lw_matvec call per mat-vec (%d launches per step), q/k/v and "
                                                    "gate/up on parallel graph branches" % ncalls),
             "grouped": (enqueue_grouped, len(groups),
                         "one lw_matvec_sequence_batch call per step: one launch of the batched kernel per group of mat-vecs that "
                         "share their activations (q/k/v together, gate/up together, the rest alone: %d per step)" % len(groups))}
    if batch > 1:
        to_time = ["per-call", "grouped"] if args.issue == "auto" else [args.issue]
    elif args.issue == "auto":
        to_time = ["launches", "persistent"]
    else:
        to_time = [args.issue]

    replays, timings = {}, {}
    for mode in to_time:
        replays[mode] = capture(torch, modes[mode][0], not args.no_graph)
        torch.cuda.synchronize()
        if lw.device_status() != 0:
            raise RuntimeError("device fault recorded during warm-up (%s)" % mode)
    # untimed look at every mode, to pick the headline before the clock sampler starts
    for mode in to_time:
        timings[mode] = timer.time(replays[mode], max(5, args.steps // 4), args.warmup)
    headline = min(to_time, key=lambda m: timings[m])
    one_step = replays[headline]
    launches_per_step = modes[headline][1]
    mma_possible = batch > 1 and fmt in MMA_FORMATS and all(c % 256 == 0 for _, _, c in shapes)
    if mma_possible and (headline == "grouped" or batch >= 3):
        # the tensor-core kernel adds into Y: with overlap one small kernel per call clears the call's Y first
        # (chained by programmatic dependent launch); without, the main kernel clears it itself
        launches_per_step += 0 if overlap_level == 0 else (len(groups) if headline == "grouped" else ncalls)

    # ---- device-resident timing of the headline mode, clocks sampled during it
    for _ in range(max(3, args.warmup)):
        one_step()
    timer.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    timer.barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        one_step()
    ev1.record(stream)
    timer.barrier()
    ms = ev0.elapsed_time(ev1)
    t_end = time.time() + 1.0               # keep the GPU busy a little longer so the sampler sees the loaded state
    while time.time() < t_end:
        one_step()
    torch.cuda.synchronize()
    clocks = sampler.stop()

    def describe(mode, ms_step):
        return {"issue": modes[mode][2], "ms_per_step": round(ms_step, 5),
                "value": round((wbytes + abytes) / (ms_step * 1e-3) / 1e9, 1), "unit": "GB/s",
                "tok_per_s": round(1e3 / ms_step, 2)}

    others = {}
    for mode in to_time:
        if mode != headline:
            others[mode] = describe(mode, timer.time(replays[mode], args.steps, 3))
    if batch == 1 and "per-call" not in to_time and not args.only and not args.no_graph:
        others["per-call"] = describe("per-call", timer.time(capture(torch, enqueue_per_call), args.steps, 3))
    if batch > 1 and all(lw.query_variant(fmt_id, r, c, batch) == lw.VARIANT_MMA for _, r, c in shapes):
        # the same step with the tensor-core kernel switched off: the fp32 tile kernel where it applies (passes of 8
        # and 4 columns), else what the heuristics would pick without it
        lw.set_variant(lw.VARIANT_TILE)
        kinds = {lw.query_variant(fmt_id, r, c, batch) for _, r, c in shapes}
        d = describe("per-call", timer.time(capture(torch, enqueue_per_call, not args.no_graph), args.steps, 3))
        d["issue"] = "per-call, tensor cores off (LW_VARIANT_TILE forced; variants launched: %s)" % sorted(kinds)
        others["fp32_only"] = d
        lw.set_variant(lw.VARIANT_AUTO)

    # ---- end to end through the host-buffer entry points of the C ABI, pinned host memory on both sides, the
    # copies inside the timed region.  Batch 1: ONE lw_matvec_sequence_host call per step (the step's activation
    # block in, the chain in the headline mode, the result block out; copies in pieces beside the kernels).  Beside it
    # (and alone for batch > 1): one lw_matvec_host call per mat-vec, each with its own two copies.
    def enqueue_host(stream):
        for i, (_, r, c) in enumerate(shapes):
            lw.matvec_host(fmt_id, wptr + offs[i], r, c, xhptr + 4 * xoffs[i], yhptr + 4 * yoffs[i],
                           xptr + 4 * xoffs[i], yptr + 4 * yoffs[i], batch, stream)

    def enqueue_seq_host(stream):
        lw.set_sequence_mode(lw.SEQ_PERSISTENT if headline == "persistent" else lw.SEQ_LAUNCHES)
        lw.matvec_sequence_host(fmt_id, seq_arr, xhptr, xptr, 4 * xt, yptr, yhptr, 4 * yt, seq_ws, stream=stream)

    ms_percall_host = timer.time(capture(torch, enqueue_host, not args.no_graph), max(3, args.steps // 5), 3)
    if batch == 1:
        ms_host = timer.time(capture(torch, enqueue_seq_host, not args.no_graph), args.steps, 3) * args.steps
        h2d, d2h = 4 * xt, 4 * yt
        e2e_path = "one lw_matvec_sequence_host call per step: the step's %d-byte activation block from pinned host " \
                   "memory to the device, the chain (%s), the %d-byte result block back to pinned host memory; the " \
                   "library moves both blocks in pieces on its own copy streams beside the kernels (a launch waits " \
                   "for the pieces it reads; a piece of results leaves when no later mat-vec writes into it)" % (
                       4 * xt, headline, 4 * yt)
    else:
        # batch > 1: the host-buffer form of the batched chain
        def enqueue_block_host(stream):
            lw.matvec_sequence_batch_host(fmt_id, seq_arr, batch, xhptr, xptr, 4 * xt, yptr, yhptr, 4 * yt, stream)
        ms_host = timer.time(capture(torch, enqueue_block_host, not args.no_graph), args.steps, 3) * args.steps
        h2d, d2h = 4 * xt, 4 * yt
        e2e_path = "one lw_matvec_sequence_batch_host call per step: the step's %d-byte activation block from pinned host " \
                   "memory to the device, the chain (one grouped call per group), the %d-byte result block back to " \
                   "pinned host memory; the library moves both blocks in pieces on its own copy streams beside the " \
                   "kernels" % (4 * xt, 4 * yt)
    lw.set_sequence_mode(lw.SEQ_AUTO)
    if lw.device_status() != 0:
        raise RuntimeError("device fault recorded during the timed region")

    ceiling = read_only_ceiling(lw, timer, W, total) if not args.only else None
    ms, ms_host = dist_util.max_over_ranks([ms, ms_host], device="cuda")

    step_ms = ms / args.steps
    total_bytes = (wbytes + abytes) * world
    gbs = total_bytes / (step_ms * 1e-3) / 1e9
    per_gpu_gbs = gbs / world
    kernel = ("matvec_seq_kernel" if headline == "persistent" else "matvec_stream_kernel") + \
        "<%s%s>" % ("Idot_" if fmt != "f16" else "", fmt)
    if batch > 1 and fmt in MMA_FORMATS and (headline == "grouped" or batch >= 3) and all(c % 256 == 0 for _, _, c in shapes):
        kernel = "matvec_mma_kernel<%s, %d>" % (fmt, 1 if batch <= 8 else 2)
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
        "dtype": arithmetic_of(fmt, batch),
        "data": "synthetic",
        "config": {
            "workload": "%s: %d mat-vecs per decode step, batch %d, weights %.3f GB in %s, fp32 activations; %s%s%s" % (
                args.workload, ncalls, batch, wbytes / 1e9, fmt, modes[headline][2],
                "" if args.no_graph else ", replayed as one CUDA graph",
                "" if (args.no_overlap or headline != "per-call") else ", programmatic dependent launch between calls"),
            "format": fmt, "batch": batch, "calls_per_step": ncalls, "issue": headline,
            "weight_bytes": wbytes, "activation_bytes": abytes,
            "l2": "weight set is %.0fx the 126 MB L2 and is streamed evict-first; no flush needed" % (wbytes / 126e6),
            "parallelism": "replicas only (one independent decode step per GPU)" if world > 1 else "single GPU",
        },
        "tok_per_s": round(world * 1e3 / step_ms, 2),
        "pct_of_nominal_8TBs": round(100 * per_gpu_gbs / NOMINAL_PEAK_GBS, 2),
        "effective_gflops": round(world * sum(2.0 * r * c * batch for _, r, c in shapes) / (step_ms * 1e-3) / 1e9, 1),
        "clocks": clocks,
        "gpu_launches": args.steps * launches_per_step,
        "other_issue_modes": others,
        "e2e": {
            "value": round((wbytes + abytes) * world / (ms_host / args.steps * 1e-3) / 1e9, 1),
            "unit": "GB/s",
            "ms_per_step": round(ms_host / args.steps, 5),
            "tok_per_s": round(world * args.steps * 1e3 / ms_host, 2),
            "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h),
            "path": e2e_path + ("" if args.no_graph else ", replayed as one CUDA graph"),
            "per_matvec_host_calls": {
                "what": "one lw_matvec_host call per mat-vec (%d calls, each: pinned host X -> device, kernel, Y -> pinned "
                        "host): %d small copies per step, bound by copy-engine latency" % (ncalls, 2 * ncalls),
                "ms_per_step": round(ms_percall_host, 5),
                "value": round((wbytes + abytes) / (ms_percall_host * 1e-3) / 1e9, 1), "unit": "GB/s",
                "h2d_bytes_per_step": int(sum(4 * batch * c for _, _, c in shapes)),
                "d2h_bytes_per_step": int(sum(4 * batch * r for _, r, _ in shapes))},
        },
        "roofline": roofline_block(
            per_gpu_gbs, kernel, (wbytes + abytes) / launches_per_step,
            int(TRAFFIC_RATIO[args.workload] * (wbytes + abytes) / launches_per_step)
            if args.workload in TRAFFIC_RATIO and batch == 1 else None, ceiling),
    }
    mma_served = batch > 1 and all(lw.query_variant(fmt_id, r, c, batch) == lw.VARIANT_MMA for _, r, c in shapes)
    if mma_served:
        # the tensor-core kernel: every weight-column product is issued twice (one per bf16 term of the
        # activation), in groups of eight columns; state the tensor work against the measured bf16 GEMM peak
        cols8 = 8 * ((batch + 7) // 8)
        issued = sum(2.0 * r * c * cols8 * 2 for _, r, c in shapes)
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
                tpeak, tsrc = float(json.load(fh)["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json bf16_tflops_sustained)"
        except Exception:
            tpeak, tsrc = 1400.0, "fallback (1.4 PFLOP/s sustained, earlier measurement on this pool)"
        result["roofline_tensor"] = {
            "bound": "tensor", "achieved": round(issued / (step_ms * 1e-3) / 1e12, 1), "peak": tpeak, "peak_source": tsrc,
            "unit": "TFLOP/s", "frac": round(issued / (step_ms * 1e-3) / 1e12 / tpeak, 4),
            "what": "bf16 products issued (2 terms x columns rounded up to 8) over the step time; the peak is the tcgen05 "
                    "GEMM figure, which the warp-level mma used here cannot reach (measured: one m16n8k16 per ~10 cycles "
                    "per SM sub-partition, i.e. about 470 TFLOP/s for the whole GPU); the HBM roofline in `roofline` is the "
                    "bound a faster contraction would hit first"}
    elif batch > 1:
        # the binding bound from batch 2 on is instruction issue, not HBM: state it with its derivation
        flops = sum(2.0 * r * c * batch for _, r, c in shapes)
        alu_peak = 148 * 128 * 1.965e9 * 2 / 1e12
        result["roofline_alu"] = {
            "bound": "alu", "achieved": round(flops / (step_ms * 1e-3) / 1e12, 2), "peak": round(alu_peak, 1),
            "unit": "TFLOP/s", "frac": round(flops / (step_ms * 1e-3) / 1e12 / alu_peak, 4),
            "derivation": "148 SMs x 128 fp32 lanes x 1.965 GHz x 2 flop per FMA = 74.4 TFLOP/s of plain FMA issue; "
                          "the integer-dot form needs 3 dp4a per 4 weight-columns on a half-rate pipe (about 50)"}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline_leg(shapes, fmt, fmt_id, batch, seed, std, outlier_p, keep_host, xh,
                                                  xoffs, Y, yoffs, args.cpu_seconds)
    if rank == 0:
        print(json.dumps(result), flush=True)
    dist_util.shutdown()


# --------------------------------------------------------- oracle legs (CPU, rank 0) ---

def cpu_baseline_leg(shapes, fmt, fmt_id, batch, seed, std, outlier_p, keep_host, xh, xoffs, Y_dev, yoffs,
                     seconds):
    """Times the oracle (as it stands) on a bounded sample of the step -- whole matrices, regenerated
    from the seeded recipe and quantised by the oracle's own quantiser -- once on all cores and once
    single-threaded, and checks the GPU results of those matrices against it with the mat-vec tolerance."""
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
    single_time, single_bytes, single_w = 0.0, 0, 0
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
        if single_time < seconds / 2:           # single-threaded: the first rows of the same matrix
            rr = max(1, min(r, int(2.0e7 // c)))
            t = time.time()
            oracle.matvec(fmt_id, blocks[:oracle.row_bytes(fmt_id, c) * rr], rr, c, x, batch, nthreads=1)
            single_time += time.time() - t
            single_bytes += int(rr * c * BYTES_PER_WEIGHT[fmt]) + 4 * batch * (rr + c)
            single_w += rr * c
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
        "single_thread": {"value": round(single_bytes / max(single_time, 1e-9) / 1e9, 4), "unit": "GB/s", "cores": 1,
                          "sample": "the first rows (up to 2e7 weights) of the first of those matrices, %.2f%% of the "
                                    "step's weights, %.1f s" % (100.0 * single_w / total_w, single_time),
                          "tok_per_s_equiv": round(1.0 / (max(single_time, 1e-9) * total_w / max(single_w, 1)), 6)},
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

    reference_line(args, METRIC, step, nbytes,
                   "first %d rows of each of the first layer's 7 matrices (%d weights = %.3f%% of a step) per step" % (
                       args.ref_rows, nweights, 100.0 * nweights / sum(r * c for _, r, c in shapes)),
                   {"format": fmt, "batch": batch},
                   extra={"tok_per_s_fraction": nweights / sum(r * c for _, r, c in shapes)})


def reference_line(args, metric, step, nbytes, sample_txt, config_extra, extra=None):
    """Times `step` (the oracle on a bounded sample) and prints the reference arm's JSON line."""
    cores = os.cpu_count() or 1
    for _ in range(max(1, args.warmup)):
        step()
    t = time.time()
    for _ in range(args.steps):
        step()
    dt = (time.time() - t) / args.steps
    gbs = nbytes / dt / 1e9
    line = {
        "impl": "reference", "metric": metric, "value": round(gbs, 4), "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": max(1, args.warmup),
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": dict({"workload": "%s (CPU oracle on a bounded sample: %s)" % (args.workload, sample_txt)}, **config_extra),
        "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    if extra and "tok_per_s_fraction" in extra:
        line["tok_per_s"] = round(extra["tok_per_s_fraction"] / dt, 5)
    print(json.dumps(line), flush=True)


# ------------------------------------------- one small mat-vec: hot and cold (config 1) ---

SINGLE_METRIC = "single mat-vec (q8_0 2048x2048, batch 1): HBM GB/s cold, microseconds per call hot and cold"


def single_spec():
    return FMT_ID["q8_0"], 2048, 2048, 64, 1       # format, rows, cols, copies, seed


def run_single(args):
    """Config 1: W 2048x2048 q8_0, x 2048.  Launch-latency-bound by construction (4.46 MB per call), so two figures:
    hot = the same matrix again and again (L2-resident), cold = rotating over 64 copies (285 MB, 2.3x the L2)."""
    torch, dist_util, lw, rank, local_rank, world = device_setup()
    fmt_id, rows, cols, copies, seed = single_spec()
    timer = Timer(torch, dist_util)
    w32 = synth.weights(seed, 0, rows, cols, 0.02, 0.0)
    blocks = lw.quantize(fmt_id, w32)
    nb = blocks.size
    stride = (nb + 255) & ~255
    W = torch.empty(copies * stride, dtype=torch.uint8, device="cuda")
    for k in range(copies):
        W[k * stride:k * stride + nb].copy_(torch.from_numpy(blocks))
    x_np = synth.activations(seed, 0, 1, cols)
    X_host = torch.from_numpy(x_np.copy()).pin_memory()
    Y_host = torch.empty(copies, rows, dtype=torch.float32).pin_memory()
    X = X_host.cuda()
    Y = torch.zeros(copies, rows, dtype=torch.float32, device="cuda")
    lw.set_overlap(not args.no_overlap)
    wp, xp, yp = W.data_ptr(), X.data_ptr(), Y.data_ptr()

    def enqueue_cold(stream):
        for k in range(copies):
            lw.matvec(fmt_id, wp + k * stride, rows, cols, xp, yp + 4 * rows * k, 1, stream)

    def enqueue_hot(stream):
        for k in range(copies):
            lw.matvec(fmt_id, wp, rows, cols, xp, yp, 1, stream)

    seq = lw.seq_items([(wp + k * stride, rows, cols, xp, yp + 4 * rows * k, lw.SEQ_DEPENDENT) for k in range(copies)])
    seq_ws = torch.zeros(64, dtype=torch.int32, device="cuda")

    def enqueue_seq(stream):
        lw.set_sequence_mode(lw.SEQ_PERSISTENT)
        lw.matvec_sequence(fmt_id, seq, seq_ws, stream=stream)
        lw.set_sequence_mode(lw.SEQ_AUTO)

    def enqueue_host(stream):
        for k in range(copies):
            lw.matvec_host(fmt_id, wp + k * stride, rows, cols, X_host.data_ptr(), Y_host.data_ptr() + 4 * rows * k,
                           xp, yp + 4 * rows * k, 1, stream)

    cold, hot, seqr, host = (capture(torch, f, not args.no_graph) for f in (enqueue_cold, enqueue_hot, enqueue_seq, enqueue_host))
    # parity of every copy's result against the oracle before timing
    parity = None
    if rank == 0 and not args.no_cpu_baseline:
        import oracle
        cold()
        torch.cuda.synchronize()
        y_ref, s_ref = oracle.matvec(fmt_id, oracle.quantize(fmt_id, w32), rows, cols, x_np, 1, nthreads=os.cpu_count() or 1)
        got = Y.cpu().numpy().astype(np.float64)
        parity = float((np.abs(got - y_ref) / (1e-4 * s_ref + 1e-6)).max())
        if not parity <= 1.0:
            raise RuntimeError("parity check failed: worst error / tolerance = %.3g" % parity)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    ms_cold = timer.time(cold, args.steps, args.warmup)
    ms_hot = timer.time(hot, args.steps, args.warmup)
    ms_seq = timer.time(seqr, args.steps, args.warmup)
    ms_host = timer.time(host, args.steps, 3)
    t_end = time.time() + 0.7
    while time.time() < t_end:
        cold()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if lw.device_status() != 0:
        raise RuntimeError("device fault recorded during the timed region")
    ms_cold, ms_hot, ms_seq, ms_host = dist_util.max_over_ranks([ms_cold, ms_hot, ms_seq, ms_host], device="cuda")
    call_bytes = nb + 4 * (rows + cols)
    step_b = copies * call_bytes
    gbs = world * step_b / (ms_cold * 1e-3) / 1e9
    result = {
        "metric": SINGLE_METRIC, "value": round(gbs, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": round(ms_cold, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": arithmetic_of("q8_0", 1), "data": "synthetic",
        "config": {"workload": "q8_0_2048: one step = %d lw_matvec calls, one per copy of a 2048x2048 q8_0 matrix "
                               "(4,456,448 bytes each; %d copies = %.0f MB, %.1fx the 126 MB L2, so every call reads cold "
                               "weights), batch 1, consecutive calls on one stream with programmatic dependent launch%s" % (
                                   copies, copies, copies * nb / 1e6, copies * nb / 126e6,
                                   "" if args.no_graph else ", replayed as one CUDA graph"),
                   "format": "q8_0", "batch": 1, "calls_per_step": copies, "weight_bytes": copies * nb,
                   "l2": "rotation over %d copies (%.1fx the L2)" % (copies, copies * nb / 126e6)},
        "us_per_call_cold": round(1e3 * ms_cold / copies, 3),
        "us_per_call_hot_l2": round(1e3 * ms_hot / copies, 3),
        "hot_l2": {"what": "the same matrix %d times in a row (L2-resident after the first call)" % copies,
                   "value": round(step_b / (ms_hot * 1e-3) / 1e9, 1), "unit": "GB/s of algorithmic bytes (served by L2)"},
        "sequence": {"what": "the same %d cold calls as ONE persistent lw_matvec_sequence kernel (each item dependent on the previous one)" % copies,
                     "us_per_call": round(1e3 * ms_seq / copies, 3), "value": round(step_b / (ms_seq * 1e-3) / 1e9, 1),
                     "unit": "GB/s"},
        "floor_us_per_call": {"at_measured_peak": round(call_bytes / measured_peak()[0] / 1e3, 3),
                              "at_nominal_8000": round(call_bytes / 8000.0 / 1e3, 3)},
        "clocks": clocks, "gpu_launches": args.steps * copies,
        "parity_worst_error_over_tolerance": None if parity is None else round(parity, 4),
        "e2e": {"value": round(world * step_b / (ms_host * 1e-3) / 1e9, 1), "unit": "GB/s",
                "ms_per_step": round(ms_host, 5), "us_per_call": round(1e3 * ms_host / copies, 3),
                "h2d_bytes_per_step": copies * 4 * cols, "d2h_bytes_per_step": copies * 4 * rows,
                "path": "one lw_matvec_host call per mat-vec (pinned host X in, pinned host Y out)"},
        "roofline": roofline_block(gbs / world, "matvec_stream_kernel<Idot_q8_0>", call_bytes, None),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        ob = oracle.quantize(fmt_id, w32)
        cores = os.cpu_count() or 1
        leg = {}
        for name, nthr in (("all_cores", cores), ("single_thread", 1)):
            reps, t = 0, time.time()
            while reps < 1 or time.time() - t < args.cpu_seconds / 2:
                oracle.matvec(fmt_id, ob, rows, cols, x_np, 1, nthreads=nthr)
                reps += 1
            dt = (time.time() - t) / reps
            leg[name] = {"value": round(call_bytes / dt / 1e9, 4), "unit": "GB/s", "cores": nthr,
                         "us_per_call": round(dt * 1e6, 1), "repetitions": reps}
        result["cpu_baseline"] = {"value": leg["all_cores"]["value"], "unit": "GB/s", "cores": cores, "kind": "oracle",
                                  "sample": "the whole 2048x2048 mat-vec, %d repetitions" % leg["all_cores"]["repetitions"],
                                  "us_per_call": leg["all_cores"]["us_per_call"], "single_thread": leg["single_thread"]}
    if rank == 0:
        print(json.dumps(result), flush=True)
    dist_util.shutdown()


def run_single_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    fmt_id, rows, cols, copies, seed = single_spec()
    ob = oracle.quantize(fmt_id, synth.weights(seed, 0, rows, cols, 0.02, 0.0))
    x = synth.activations(seed, 0, 1, cols)
    cores = os.cpu_count() or 1
    reference_line(args, SINGLE_METRIC, lambda: oracle.matvec(fmt_id, ob, rows, cols, x, 1, nthreads=cores),
                   ob.size + 4 * (rows + cols), "one 2048x2048 q8_0 mat-vec per step (1 of the GPU arm's %d calls per step)" % copies,
                   {"format": "q8_0", "batch": 1})


# ------------------------------------------------------------ stand-alone dequantisation ---

DEQUANT_METRIC = "stand-alone dequantisation: HBM GB/s of (block bytes read + 4 bytes written) per weight"
DEQUANT_WEIGHTS = 1 << 28


def run_dequant(args):
    """One step = one lw_dequant call over 2^28 weights (1 GiB of fp32 out, 8x the L2)."""
    torch, dist_util, lw, rank, local_rank, world = device_setup()
    fmt = args.workload[len("dequant_"):]
    fmt_id = FMT_ID[fmt]
    n = DEQUANT_WEIGHTS
    timer = Timer(torch, dist_util)
    nb = lw.row_bytes(fmt_id, n)
    # blocks: a seeded 16 Mi-weight tile quantised on the host and repeated (timing depends on bytes, not values)
    tile_n = 1 << 24
    tile = lw.quantize(fmt_id, synth.normal(77, fmt_id, tile_n, 0.02, 0.01))
    W_host = torch.from_numpy(np.tile(tile, n // tile_n)).pin_memory()
    W = W_host.cuda()
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    out_host = torch.empty(n, dtype=torch.float32).pin_memory()
    step = lambda: lw.dequant(fmt_id, W, n, out)
    step()
    torch.cuda.synchronize()
    parity = None
    if rank == 0 and not args.no_cpu_baseline:
        import oracle
        m = 1 << 20
        want = oracle.dequant(fmt_id, oracle.quantize(fmt_id, synth.normal(77, fmt_id, tile_n, 0.02, 0.01))[:oracle.row_bytes(fmt_id, m)], m)
        for start in (0, n - tile_n):                 # first and last tile: the first 2^20 weights of each, bit for bit
            got = out[start:start + m].cpu().numpy()
            if not (got.view(np.uint32) == want.view(np.uint32)).all():
                raise RuntimeError("dequant parity failed at %d" % start)
        parity = True
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    ms = timer.time(step, args.steps, args.warmup)
    t_end = time.time() + 0.7
    while time.time() < t_end:
        step()
    torch.cuda.synchronize()
    clocks = sampler.stop()

    def e2e_step():
        W.copy_(W_host, non_blocking=True)
        step()
        out_host.copy_(out, non_blocking=True)

    ms_e2e = timer.time(e2e_step, max(2, args.steps // 10), 3)
    ms, ms_e2e = dist_util.max_over_ranks([ms, ms_e2e], device="cuda")
    step_b = nb + 4 * n
    gbs = world * step_b / (ms * 1e-3) / 1e9
    result = {
        "metric": DEQUANT_METRIC, "value": round(gbs, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": round(ms, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bytes -> f32, bit-exact decode", "data": "synthetic",
        "config": {"workload": "%s: one lw_dequant call over 2^28 weights per step (%.3f GB of %s blocks in, 1.074 GB of "
                               "fp32 out; the output alone is 8.5x the 126 MB L2)" % (args.workload, nb / 1e9, fmt),
                   "format": fmt, "weights": n, "bytes_per_weight": BYTES_PER_WEIGHT[fmt] + 4,
                   "l2": "input + output are %.1fx the L2; streaming stores" % (step_b / 126e6)},
        "weights_per_s": round(world * n / (ms * 1e-3), 1), "clocks": clocks, "gpu_launches": args.steps,
        "parity_bit_exact_on_samples": parity,
        "e2e": {"value": round(world * step_b / (ms_e2e * 1e-3) / 1e9, 1), "unit": "GB/s", "ms_per_step": round(ms_e2e, 4),
                "h2d_bytes_per_step": int(nb), "d2h_bytes_per_step": int(4 * n),
                "path": "blocks from pinned host memory in, lw_dequant, fp32 result back to pinned host memory (PCIe-bound)"},
        "roofline": roofline_block(gbs / world, ("dequant_q45k_kernel<%s>" if fmt in ("q4_K", "q5_K") else "dequant_warp_kernel<%s>") % fmt, step_b, None),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        m = 1 << 22
        ob = oracle.quantize(fmt_id, synth.normal(77, fmt_id, m, 0.02, 0.01))
        reps, t = 0, time.time()
        while reps < 1 or time.time() - t < args.cpu_seconds:
            oracle.dequant(fmt_id, ob, m)
            reps += 1
        dt = (time.time() - t) / reps
        result["cpu_baseline"] = {"value": round((ob.size + 4 * m) / dt / 1e9, 4), "unit": "GB/s", "cores": 1, "kind": "oracle",
                                  "sample": "2^22 weights (1.6%% of a step) per repetition, %d repetitions" % reps}
    if rank == 0:
        print(json.dumps(result), flush=True)
    dist_util.shutdown()


def run_dequant_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    fmt = args.workload[len("dequant_"):]
    fmt_id = FMT_ID[fmt]
    m = 1 << 22
    ob = oracle.quantize(fmt_id, synth.normal(77, fmt_id, m, 0.02, 0.01))
    reference_line(args, DEQUANT_METRIC, lambda: oracle.dequant(fmt_id, ob, m), ob.size + 4 * m,
                   "2^22 weights (1.6% of the GPU arm's step) per step", {"format": fmt})


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
        "vs_baseline": None, "dtype": "f32 in/out; f16 tensor-core products of exact cache codes with the query and the "
                                       "probabilities as high + low f16 pairs, fp32 accumulation and softmax"
        if variant == 2 else "f32 in/out; exact block decode, fp32 FMA", "data": "synthetic",
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


def spawn_ranks(args):
    """`python bench.py --gpus N` without a torchrun environment: start the N ranks here (one per GPU)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_q4_K",
                    choices=sorted(synth.WORKLOADS) + sorted(synth.ATTN_WORKLOADS) + list(SINGLE_WORKLOADS) +
                    list(DEQUANT_WORKLOADS))
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=None, help="use fewer layers (debugging only)")
    ap.add_argument("--only", default=None, help="comma-separated substrings: keep only matching mat-vecs "
                                                  "(profiling of single kernels)")
    ap.add_argument("--issue", default="auto", choices=["auto", "launches", "persistent", "per-call", "grouped"],
                    help="how the step is issued (auto: batch 1 times launches and persistent, batch > 1 per-call and grouped; the faster is the headline)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--serial", action="store_true", help="per-call mode on one branch: every mat-vec waits for the previous one")
    ap.add_argument("--no-overlap", action="store_true")
    ap.add_argument("--overlap", type=int, default=None, choices=[0, 1, 2],
                    help="lw_set_overlap level (default 1 at batch 1, 2 beyond: weights are parameters nothing on the stream writes)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=4.0)
    ap.add_argument("--ref-rows", type=int, default=512)
    ap.add_argument("--tuning-table", default=None, help="per-shape table written by the autotune sweep, installed before the run")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        spawn_ranks(args)
    attn = args.workload in synth.ATTN_WORKLOADS
    single = args.workload in SINGLE_WORKLOADS
    deq = args.workload in DEQUANT_WORKLOADS
    if args.impl == "reference":
        (run_attn_reference if attn else run_single_reference if single else run_dequant_reference if deq else run_reference)(args)
    else:
        (run_attn if attn else run_single if single else run_dequant if deq else run_step)(args)


if __name__ == "__main__":
    main()
