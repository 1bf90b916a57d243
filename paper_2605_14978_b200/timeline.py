"""Per-warp timeline of the bulk-copy row kernel: ``PPOW_LIBRARY=timeline python -m paper_2605_14978_b200.timeline
[workload[:windows] ...]``.

Runs the scoring pass of each workload on the timeline build of the library (every warp records when it
started, when its first tile arrived, when it ended, how many items and tiles it did and how many cycles it
spent waiting for copies and in item ends) and prints, per workload: the ramp (start to first data), the spread
of the warps' end times (the tail), the split of a warp's cycles, and the delivered bandwidth over 40 slices of
the launch.  This is how the work plan and the pipeline prologue of the kernel were tuned.
"""
import os
import sys

import numpy as np
import torch

from . import binding as B
from . import build as build_mod
from . import workloads as W


def run(w, label, dev):
    mode = B.PPOW_GREEDY if w.modes[-1] == "greedy" else B.PPOW_STOCHASTIC
    x = W.generate(w, dev)
    params = B.make_params(w.N, w.K, w.V, B.DTYPE_CODES[w.torch_dtype], mode, w.c, w.temperature)
    out = B.alloc_outputs(w.N, w.K, dev)
    ws = B.alloc_workspace(B.ppow_score_workspace_bytes(params), dev)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(6):
        B.ppow_score_windows_traced(params, x["draft_logits"], x["target_logits"], x["draft_tokens"], x["uniforms"],
                                    x["valid_len"], None, out, ws, stream, e0, e1)
    torch.cuda.synchronize()
    event_us = e0.elapsed_time(e1) * 1e3
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    warps = sms * 2 * 8
    status, t = B.ppow_timeline_read(warps)
    if status != B.PPOW_OK:
        raise SystemExit("not the timeline build: run with PPOW_LIBRARY=timeline")
    t = t.astype(np.int64)
    t = t[t[:, 2] > 0]
    t0, t1, t2, items, tiles, sm, wait, endc, total, reduce, opened = (t[:, i] for i in range(11))
    base = t0.min()
    span = (t2.max() - base) / 1e3
    rows = int(x["valid_len"].sum()) if x["valid_len"] is not None else w.N * w.K
    nbytes = 2 * rows * w.V * (4 if w.dtype == "f32" else 2)
    q = lambda a: np.percentile(a, [0, 10, 50, 90, 100]).round(2).tolist()
    print("== %s: %d warps, row kernel %.1f us by events, %.1f us first start to last end, %.3f GB -> %.0f GB/s by events"
          % (label, len(t), event_us, span, nbytes / 1e9, nbytes / event_us / 1e3))
    print("   percentiles 0/10/50/90/100 over warps")
    print("   start to first data, us      ", q((t1 - t0) / 1e3))
    print("   end after first start, us    ", q((t2 - base) / 1e3))
    print("   items per warp               ", q(items), "  tiles per warp", q(tiles))
    print("   share of cycles waiting      ", q(wait / total), "  in item ends", q(endc / total))
    print("   cycles per item end          ", q(endc / np.maximum(items, 1)), "  cycles per tile", q((total - endc) / np.maximum(tiles, 1)))
    it = np.maximum(items, 1)
    print("   of an item end: up to the end of the warp reduction", q(reduce / it), "  reset + next item", q(opened / it),
          "  argmax index + store", q((endc - reduce - opened) / it))
    grid = np.linspace(0, span, 41)
    done = [(np.clip((base + g * 1e3 - t1) / np.maximum(t2 - t1, 1), 0, 1) * tiles).sum() for g in grid]
    tile_bytes = 2 * 128 * 16
    rate = np.diff(done) * tile_bytes / (np.diff(grid) * 1e-6) / 1e12
    print("   TB/s per 1/40 of the launch   " + " ".join("%.1f" % r for r in rate))
    print("   warps still running 20/10/5/2 us before the end:", [int((t2 > base + (span - d) * 1e3).sum()) for d in (20, 10, 5, 2)])


def main(argv):
    if os.environ.get("PPOW_LIBRARY") != "timeline":
        raise SystemExit("run as: PPOW_LIBRARY=timeline python -m paper_2605_14978_b200.timeline [workload[:windows] ...]")
    build_mod.build(timeline=True)
    dev = torch.device("cuda:0")
    specs = argv or ["vicuna_like", "llama3_like:256", "llama3_like:1024"]
    for spec in specs:
        name, _, n = spec.partition(":")
        w = W.BY_NAME[name]
        if n:
            w = W.scaled(w, int(n), name=w.name)
        run(w, spec, dev)


if __name__ == "__main__":
    main(sys.argv[1:])
