#!/usr/bin/env python
"""Benchmark of the PPOW window-scoring pass.

One step = one pass of the whole hot path over one batch of synthetic windows: the fused row
reduction over both logit tensors, the per-window scan (acceptance, accepted length, rewards, window
score) and the ADAW top-fraction selection.  Default workload: the Llama-3-like configuration
(N=2048 windows, K=8, V=128256, bf16 logits, stochastic acceptance at T=1, c=0.04, keep 25 %).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ppow|reference] [--workload NAME]

Prints one JSON line (rank 0).  With --gpus N > 1 (launched under torch.distributed.run) every rank
scores its own N windows; the window scores are all-gathered and every rank selects over the global
score array (weak scaling).  --impl reference times the float64 CPU oracle instead.
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

import torch

from paper_2605_14978_b200 import workloads as W

METRIC = "windows/s and logit GB/s (% of B200 HBM peak) at V=128256, K=8, N=2048"
# DRAM bytes (read + write) per window of the row-reduction kernel from the ncu capture summarised in
# profiles/row_reduce_pipe_bf16_llama3_like.md (256-window case; traffic grows in proportion to the
# windows processed).  Only valid for that kernel on that workload shape.
NCU_TRAFFIC_BYTES_PER_WINDOW = {"llama3_like": 4145686.7}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ppow", choices=["ppow", "reference"])
    ap.add_argument("--workload", default="llama3_like", choices=[w.name for w in W.WORKLOADS])
    ap.add_argument("--mode", default=None, choices=[None, "greedy", "stochastic"])
    ap.add_argument("--windows", type=int, default=None, help="override N (small cases for profiler captures)")
    ap.add_argument("--logits", default=None, choices=[None, "bf16", "f32", "f16"],
                    help="override the storage type of the logits (same recipe, rounded once to that type)")
    ap.add_argument("--train", action="store_true",
                    help="the step also produces the training-side quantities: KL(Q||P), nabla and the softmax "
                         "normalisers from the scoring pass, the group-relative advantage (groups of 8), and the "
                         "expected-acceptance pass (a second read of both logit tensors)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(n_gpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        if torch.cuda.is_available():
            torch.cuda.set_device(local)
        dist.init_process_group(backend)
    return world, rank, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value, world, device):
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def oracle_modes():
    import oracle
    return {"greedy": oracle.GREEDY, "stochastic": oracle.STOCHASTIC}


def time_oracle(w, mode, x_host, n_threads):
    import oracle
    t0 = time.perf_counter()
    o = oracle.score_windows(x_host["draft_logits"], x_host["target_logits"], x_host["draft_tokens"],
                             mode=oracle_modes()[mode], c=w.c, temperature=w.temperature,
                             uniforms=x_host["uniforms"], valid_len=x_host["valid_len"], n_threads=n_threads)
    oracle.select_windows(o["score"], min(w.n_keep, len(o["score"])))
    return time.perf_counter() - t0


def host_sample(w, chunks, device):
    x = W.generate(w, device, chunks=chunks)
    return {k: (None if v is None else v.cpu()) for k, v in x.items()}


# -------------------------------------------------------------------------------------- reference arm


def run_reference(args):
    """Times the float64 CPU oracle (as it stands) on the machine's host cores; rank 0 only."""
    world, rank, local = int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), 0
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = W.BY_NAME[args.workload]
    mode = args.mode or w.modes[-1]
    cores = os.cpu_count() or 1
    gen_dev = torch.device("cuda:0") if torch.cuda.is_available() else torch.device("cpu")
    n_chunks = (w.N + W.CHUNK - 1) // W.CHUNK
    per_step = 1                                   # one chunk of 64 windows per step
    samples = [host_sample(w, [(i * per_step) % n_chunks], gen_dev) for i in range(min(4, n_chunks))]
    times = []
    for i in range(args.warmup + args.steps):
        dt = time_oracle(w, mode, samples[i % len(samples)], cores)
        if i >= args.warmup:
            times.append(dt)
    windows = samples[0]["draft_tokens"].shape[0]
    total = sum(times)
    value = windows * len(times) / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "windows/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "N": w.N, "K": w.K, "V": w.V, "logits": w.dtype, "mode": mode,
                   "temperature": w.temperature, "c": w.c, "n_keep": w.n_keep},
        "cpu_baseline": {"value": value, "unit": "windows/s", "cores": cores, "kind": "oracle",
                         "sample": "%d windows of %s per step (one 64-window chunk), float64 C oracle with "
                                   "pthreads" % (windows, w.name)},
        "e2e": {"value": value, "unit": "windows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# -------------------------------------------------------------------------------------- ppow arm


def run_ppow(args):
    from paper_2605_14978_b200 import binding as B
    from paper_2605_14978_b200 import build as build_mod
    from paper_2605_14978_b200 import sharding as S

    if not torch.cuda.is_available():
        raise SystemExit("bench.py --impl ppow needs a CUDA device; there is no CPU path")
    world, rank, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local if world > 1 else 0)
    torch.cuda.set_device(dev)
    if rank == 0:
        build_mod.build()
    barrier(world)
    B.load_library()

    w = W.BY_NAME[args.workload]
    if args.windows:
        w = W.scaled(w, args.windows, name=w.name)
    if args.logits:
        import dataclasses
        w = dataclasses.replace(w, dtype=args.logits)
    mode = args.mode or w.modes[-1]
    bmode = B.PPOW_GREEDY if mode == "greedy" else B.PPOW_STOCHASTIC
    n_chunks = (w.N + W.CHUNK - 1) // W.CHUNK
    # weak scaling: rank r scores windows [r*N, (r+1)*N) of a world*N-window instance of the workload
    wg = W.scaled(w, w.N * world, name=w.name)
    x = W.generate(wg, dev, chunks=range(rank * n_chunks, (rank + 1) * n_chunks))
    N, K, V = w.N, w.K, w.V
    n_total, n_keep = N * world, wg.n_keep

    params = B.make_params(N, K, V, {"f32": B.PPOW_F32, "bf16": B.PPOW_BF16, "f16": B.PPOW_F16}[w.dtype], bmode, w.c, w.temperature)
    out = B.alloc_outputs(N, K, dev)
    if args.train:
        out.update(B.alloc_train_outputs(N, K, dev))
        advantage = torch.empty((N,), dtype=torch.float32, device=dev)
        exp_accept = torch.empty((N, K), dtype=torch.float32, device=dev)
        ref_logp = torch.empty((N,), dtype=torch.float32, device=dev)
        row_logp = torch.empty((N, K), dtype=torch.float32, device=dev)
        group = 8 if N % 8 == 0 else 1
    ws = B.alloc_workspace(B.ppow_score_workspace_bytes(params), dev)
    selected = torch.empty((n_keep,), dtype=torch.int32, device=dev)
    sel_ws = B.alloc_workspace(B.ppow_select_workspace_bytes(n_total), dev)
    stream = torch.cuda.current_stream()

    acc_events, ref_events = [], []

    def step(ev0=None, ev1=None):
        B.ppow_score_windows_traced(params, x["draft_logits"], x["target_logits"], x["draft_tokens"], x["uniforms"],
                                    x["valid_len"], None, out, ws, stream, ev0, ev1)
        if args.train:
            B.ppow_group_advantage(out["reward"], group, 1e-6, advantage, stream)
            ea, eb = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) if ev0 is not None else (None, None)
            if ea is not None:
                ea.record(stream)
            B.ppow_expected_acceptance(params, x["draft_logits"], x["target_logits"], x["valid_len"], out["lse_p"],
                                       out["lse_q"], exp_accept, stream)
            if ea is not None:
                eb.record(stream)
                acc_events.append((ea, eb))
            # the target's logits stand in for the logits along its reference window (same shape and type)
            B.ppow_reference_logprob(params, x["target_logits"], x["valid_len"], row_logp, ref_logp, stream)
            if ea is not None:
                ec = torch.cuda.Event(enable_timing=True)
                ec.record(stream)
                ref_events.append((eb, ec))
        scores = S.gather_scores(out["score"], n_total) if world > 1 else out["score"]   # the one exchange step
        B.ppow_select_windows(scores, n_keep, selected, None, sel_ws, stream)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    ev_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in ev_pairs:
        a.record(), b.record()                      # create the CUDA events before the timed region
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(dev.index or 0)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier(world)
    torch.cuda.synchronize()
    start.record()
    for a, b in ev_pairs:
        step(a, b)
    stop.record()
    torch.cuda.synchronize()
    barrier(world)
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = max_over_ranks(start.elapsed_time(stop), world, dev)
    reduce_ms = [a.elapsed_time(b) for a, b in ev_pairs]
    reduce_avg_ms = max_over_ranks(sum(reduce_ms) / len(reduce_ms), world, dev)
    flags = B.ppow_read_error_flags(ws)

    valid_rows = int(x["valid_len"].sum().item()) if x["valid_len"] is not None else N * K
    esize = 4 if w.dtype == "f32" else 2
    algo_bytes = 2 * valid_rows * V * esize         # both logit tensors, read once; per launch of the row kernel
    peak, peak_kind = measured_peak()
    achieved = algo_bytes / (reduce_avg_ms * 1e-3) / 1e9

    # ---- end to end through the host-buffer entry point: pinned host inputs -> results on the host
    e2e = None
    if not args.no_e2e:
        host = {k: (None if v is None else v.cpu().pin_memory()) for k, v in x.items()}
        out_host = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in out.items()}
        sel_host = torch.empty((w.n_keep,), dtype=torch.int32).pin_memory()
        scratch = B.alloc_workspace(B.ppow_host_scratch_bytes(params, N), dev)

        def e2e_step():
            B.ppow_score_and_select_host(params, host["draft_logits"], host["target_logits"], host["draft_tokens"],
                                         host["uniforms"], host["valid_len"], None, out_host, w.n_keep, sel_host,
                                         None, scratch, stream)
            torch.cuda.synchronize()
            return int(sel_host[0])                 # the step's result is read on the host

        e2e_step()
        e2e_steps = max(1, min(args.steps, 10))
        barrier(world)
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        e2e_s = max_over_ranks(time.perf_counter() - t0, world, dev)
        h2d = sum(v.numel() * v.element_size() for v in host.values() if v is not None)
        d2h = sum(v.numel() * v.element_size() for v in out_host.values()) + sel_host.numel() * 4
        e2e = {"value": n_total * e2e_steps / e2e_s, "unit": "windows/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": 1e3 * e2e_s / e2e_steps,
               "note": "ppow_score_and_select_host: pinned host logits copied to the device inside the timed region"}
        del host, scratch

    # ---- the oracle, as it stands, on this machine's host cores (rank 0, N = 1 only)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        cores = os.cpu_count() or 1
        n_sample_chunks = min(n_chunks, 16)     # ~25 core-seconds of oracle work on the headline workload
        idx = slice(0, min(N, n_sample_chunks * W.CHUNK))
        xs = {k: (None if v is None else v[idx].cpu()) for k, v in x.items()}
        dt = time_oracle(w, mode, xs, cores)
        nw = xs["draft_tokens"].shape[0]
        cpu_baseline = {"value": nw / dt, "unit": "windows/s", "cores": cores, "kind": "oracle",
                        "sample": "first %d windows of %s, float64 C oracle with pthreads, %.1f s wall" % (nw, w.name, dt)}

    if rank != 0:
        return
    step_ms = elapsed_ms / args.steps
    value = n_total / (step_ms * 1e-3)
    line = {
        "metric": METRIC, "value": value, "unit": "windows/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "N_per_gpu": N, "K": K, "V": V, "logits": w.dtype, "mode": mode,
                   "temperature": w.temperature, "c": w.c, "n_keep": n_keep,
                   "l2": "inputs (%.2f GB per GPU) larger than L2; no flush needed" % (algo_bytes / 1e9)
                   if algo_bytes > 4e8 else "inputs fit L2: not an HBM figure"},
        "logit_gbs": world * algo_bytes / (step_ms * 1e-3) / 1e9,
        "roofline": {"bound": "hbm", "kernel": "row_reduce", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": "of " + peak_kind, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "traffic": (NCU_TRAFFIC_BYTES_PER_WINDOW[w.name] * N
                                 if w.name in NCU_TRAFFIC_BYTES_PER_WINDOW and w.dtype == "bf16" and not args.train else None),
                     "traffic_source": "ncu dram__bytes_read+write on a 256-window capture, scaled by windows",
                     "algorithmic_bytes_per_launch": algo_bytes, "kernel_ms": reduce_avg_ms},
        "training": ({"kl_rev_in_scoring_pass": True, "group_size": group,
                      "expected_acceptance_ms": sum(a.elapsed_time(b) for a, b in acc_events) / len(acc_events),
                      "expected_acceptance_gbs": algo_bytes / (sum(a.elapsed_time(b) for a, b in acc_events)
                                                               / len(acc_events) * 1e-3) / 1e9,
                      "reference_logprob_ms": sum(a.elapsed_time(b) for a, b in ref_events) / len(ref_events),
                      "reference_logprob_gbs": 0.5 * algo_bytes / (sum(a.elapsed_time(b) for a, b in ref_events)
                                                                   / len(ref_events) * 1e-3) / 1e9}
                     if args.train else None),
        "e2e": e2e, "cpu_baseline": cpu_baseline, "gpu_launches": (7 if args.train else 3) * args.steps, "clocks": clocks,
        "error_flags": flags,
    }
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ppow(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
