"""Single-device sweep of the streaming kernels' tunables over the decode shapes of the benchmark
models: worker groups per CTA, ring slots per group and ring-slot size (`lw_set_tuning`), timed per
(format, rows, cols) as back-to-back launches inside a CUDA graph with programmatic dependent launch.
Writes a Markdown table: per shape the time under the launch heuristics' own choice, the best
setting found, the ratio between the two, and the time of the other kernel family (fp32 activations
instead of the integer-dot form) where a format has both.  With --table it also writes the per-shape
table (JSON) of the settings that beat the heuristics by more than 2 %, which `lw.load_tuning_table`
installs (`lw_set_shape_tuning`) and the launch heuristics then consult.

    python -m paper_2605_20706_b200.autotune --out profiles/autotune_stream_kernels.md --table tuning_table.json

The matrices are seeded synthetic weights quantised with the library's host quantiser (a 1024-row
slab tiled to the full height: the timing depends on bytes and shapes only); enough copies of each
matrix are cycled through to keep the working set well above the 126 MB L2.
"""
from __future__ import annotations

import argparse
import itertools
import sys

import numpy as np

from . import lw, synth

GROUPS = (2, 1)
STAGES = (2, 3)
STAGE_KB = (24, 32, 40, 48, 64)


def unique_shapes(models):
    seen, out = set(), []
    for model in models:
        shapes = synth.llama_8b_shapes() if model == "8b" else synth.llama_1b_shapes()
        for name, rows, cols in shapes:
            leaf = name.split(".")[-1]
            if (rows, cols) not in seen:
                seen.add((rows, cols))
                out.append(("%s %s" % (model, leaf), rows, cols))
        # the grouped launches of a step are planned by the sum of their rows
        by_leaf = {name.split(".")[-1]: (rows, cols) for name, rows, cols in shapes}
        for label, leaves in (("q+k+v", ("q", "k", "v")), ("gate+up", ("gate", "up"))):
            rows, cols = sum(by_leaf[l][0] for l in leaves), by_leaf[leaves[0]][1]
            if (rows, cols) not in seen:
                seen.add((rows, cols))
                out.append(("%s %s" % (model, label), rows, cols))
    return out


def make_weights(torch, fmt, rows, cols, min_bytes):
    slab_rows = min(rows, 1024)
    slab = lw.quantize(fmt, synth.weights(17, fmt, slab_rows, cols, 0.02, 0.0))
    reps = -(-rows // slab_rows)
    one = np.tile(slab, reps)[: lw.row_bytes(fmt, cols) * rows]
    copies = max(2, -(-min_bytes // one.size))
    return [torch.from_numpy(one).cuda() for _ in range(copies)]


def time_setting(torch, fmt, rows, cols, ws, x, ys, launches, replays):
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(2):
            lw.matvec(fmt, ws[i % len(ws)], rows, cols, x, ys[i % len(ys)], 1, stream)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for i in range(launches):
            lw.matvec(fmt, ws[i % len(ws)], rows, cols, x, ys[i % len(ys)], 1, torch.cuda.current_stream())
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (replays * launches)      # microseconds per launch


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--formats", default="q4_K,q4_0,q8_0,f16")
    ap.add_argument("--models", default="8b,1b")
    ap.add_argument("--out", default=None)
    ap.add_argument("--table", default=None, help="write the per-shape table of winning settings (JSON) here")
    ap.add_argument("--launches", type=int, default=24)
    ap.add_argument("--replays", type=int, default=6)
    args = ap.parse_args()
    import torch

    if not torch.cuda.is_available():
        raise SystemExit("autotune needs a CUDA device")
    lw.set_overlap(True)
    lines = ["| format | matrix | rows x cols | heuristics: groups/slots/slot KB | us | best: groups/slots/slot KB | us | "
             "heuristics / best | fp32-activation family us |", "|---|---|---|---|---|---|---|---|---|"]
    grids, table = [], []
    for fname in args.formats.split(","):
        fmt = lw.FORMATS[fname]
        for label, rows, cols in unique_shapes(args.models.split(",")):
            lw.set_tuning()
            info = lw.plan_info(fmt, rows, cols)
            if info["ctas"] == 0:
                continue
            ws = make_weights(torch, fmt, rows, cols, 420 * 2 ** 20)
            x = torch.from_numpy(synth.activations(17, 0, 1, cols)).cuda()
            ys = [torch.empty(rows, dtype=torch.float32, device="cuda") for _ in range(4)]
            launches = args.launches if rows < 100000 else 8
            base = time_setting(torch, fmt, rows, cols, ws, x, ys, launches, args.replays)
            results = {}
            for g, s, kb in itertools.product(GROUPS, STAGES, STAGE_KB):
                lw.set_tuning(g, s, kb)
                got = lw.plan_info(fmt, rows, cols)
                key = (got["worker_groups"], got["stages"], got["stage_bytes"])
                if got["ctas"] == 0 or key in results:
                    continue                       # not feasible, or the same geometry as an earlier setting
                results[key] = (time_setting(torch, fmt, rows, cols, ws, x, ys, launches, args.replays), (g, s, kb))
            lw.set_tuning()
            other = None
            if fname in ("q8_0", "q4_0", "q4_K"):              # the variant is a tunable too: the fp32-activation family
                lw.set_variant(lw.VARIANT_STREAM)
                other = time_setting(torch, fmt, rows, cols, ws, x, ys, launches, args.replays)
                lw.set_variant(lw.VARIANT_AUTO)
            best_key = min(results, key=lambda k: results[k][0])
            best_us = results[best_key][0]
            if base / best_us > 1.02:
                g, s, kb = results[best_key][1]
                table.append({"format": fname, "rows": rows, "cols": cols, "worker_groups": g, "stages": s, "stage_kb": kb,
                              "us_heuristics": round(base, 2), "us_tuned": round(best_us, 2)})
            lines.append("| %s | %s | %d x %d | %d/%d/%.0f | %.2f | %d/%d/%.0f | %.2f | %.3f | %s |" % (
                fname, label, rows, cols, info["worker_groups"], info["stages"], info["stage_bytes"] / 1024, base,
                best_key[0], best_key[1], best_key[2] / 1024, best_us, base / best_us,
                "%.2f" % other if other is not None else "-"))
            grids.append((fname, label, rows, cols, results))
            print(lines[-1], file=sys.stderr, flush=True)
            del ws
            torch.cuda.empty_cache()
    if lw.device_status() != 0:
        raise SystemExit("device fault recorded during the sweep")
    text = ["# Tunables sweep of the streaming kernels (`python -m paper_2605_20706_b200.autotune`)", "",
            "Microseconds per launch, back-to-back launches of one matrix in a CUDA graph with programmatic",
            "dependent launch, working set cycled above the L2 size.  \"heuristics\" is what `make_plan` chooses",
            "on its own; \"best\" the fastest of the feasible settings of worker groups (1, 2), ring slots per",
            "group (2, 3) and ring-slot size (24..64 KB).", ""] + lines + [""]
    for fname, label, rows, cols, results in grids:
        if rows * cols not in (14336 * 4096, 4096 * 4096):
            continue
        text.append("%s, %s (%d x %d): groups/slots/slot KB -> us: " % (fname, label, rows, cols) + ", ".join(
            "%d/%d/%.0f %.2f" % (k[0], k[1], k[2] / 1024, v[0]) for k, v in sorted(results.items(), key=lambda kv: kv[1][0])))
        text.append("")
    if args.table:
        import json
        with open(args.table, "w") as fh:
            json.dump(table, fh, indent=1)
    out = "\n".join(text)
    if args.out:
        with open(args.out, "w") as fh:
            fh.write(out)
    print(out)


if __name__ == "__main__":
    main()
