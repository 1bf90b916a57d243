#!/usr/bin/env python
"""Benchmark of the PPOW window-scoring pass.

One step = one pass of the whole hot path over one batch of synthetic windows: the fused row
reduction over both logit tensors, the per-window scan (acceptance, accepted length, rewards, window
score) and the ADAW top-fraction selection.  Default workload: the Llama-3-like configuration
(N=2048 windows, K=8, V=128256, bf16 logits, stochastic acceptance at T=1, c=0.04, keep 25 %).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ppow|reference] [--workload NAME]

Prints one JSON line (rank 0).  Besides the K timed steps the line carries, at one GPU: the same step
timed for at least two seconds (the regime under the board's power limit), each regime with the SM
clocks sampled inside its own timed region; a read-only streaming pass over the same logit buffers
(the bandwidth a kernel that only reads reaches on this GPU); the float64 CPU oracle timed on a sample
of the same buffers and the element-by-element comparison of the GPU results with it; the end-to-end
number through the host-buffer entry point; and one entry per other workload.  With --gpus N > 1
(launched under torch.distributed.run) every rank scores its own N windows; the window scores are
all-gathered and every rank selects over the global score array (weak scaling).
--impl reference times the float64 CPU oracle instead.
"""
import argparse
import dataclasses
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_14978_b200 import workloads as W

METRIC = "windows/s and logit GB/s (% of B200 HBM peak) at V=128256, K=8, N=2048"
# DRAM bytes (read + write) per window of the row-reduction kernel from the ncu capture summarised in
# profiles/row_reduce_pipe_bf16_llama3_like.md (256-window case; traffic grows in proportion to the
# windows processed): mean of two launches, (1,053,934,336 read + 2,611,200 written) / 256.  Only valid for
# that kernel on that workload shape; None = not re-taken since the kernel last changed.
NCU_TRAFFIC_BYTES_PER_WINDOW = {"llama3_like": 4127131.0}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
RTOL, ATOL, BAND = 1e-4, 1e-6, 1e-6      # float tolerance and the band of the stochastic acceptance test
SUSTAINED_SECONDS = 2.0
PARITY_SAMPLE_WINDOWS = 64               # per entry of "workloads"


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
                         "normalisers from the scoring pass, the group-relative advantage (groups of 8), the "
                         "expected-acceptance pass (a second read of both logit tensors) and the reference-window "
                         "log-probability pass")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true",
                    help="skip everything that runs the oracle: its timing and the parity counts")
    ap.add_argument("--no-sustained", action="store_true", help="skip the >= 2 s regime")
    ap.add_argument("--no-workloads", action="store_true", help="skip the entries for the other workloads")
    ap.add_argument("--no-probe", action="store_true", help="skip the read-only streaming reference")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def config_of(w, mode):
    """The workload description; identical in both arms for the same command line."""
    nominal = 2 * w.N * w.K * w.V * (4 if w.dtype == "f32" else 2)
    return {"workload": w.name, "N": w.N, "K": w.K, "V": w.V, "logits": w.dtype, "mode": mode,
            "temperature": w.temperature, "c": w.c, "n_keep": w.n_keep,
            "l2": ("inputs (%.2f GB per GPU) larger than L2; no flush needed" % (nominal / 1e9)) if nominal > 4e8
            else "inputs fit L2: not an HBM figure"}


# ------------------------------------------------------------------------------------ clock sampling


class ClockSampler:
    """Samples SM clock, power and clock-event reasons (read-only NVML queries) every few milliseconds on a
    thread, with host timestamps, so that each timed region can be given the samples that fall inside it.
    Falls back to an `nvidia-smi -lms` child (samples of the whole run) when NVML cannot be loaded."""
    REASONS = ((0x4, "sw_power_cap"), (0x8, "hw_slowdown"), (0x20, "sw_thermal_slowdown"),
               (0x40, "hw_thermal_slowdown"), (0x80, "hw_power_brake_slowdown"))
    SMI_FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
                  "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                  "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.samples = []          # (t, sm_mhz, power_w, reason bits)
        self.max_mhz = None
        self.source = None
        self._stop = threading.Event()
        self._thread = None
        self._smi = None
        self._handle = None
        self._nv = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            try:
                self._handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                self._handle = pynvml.nvmlDeviceGetHandleByIndex(device.index or 0)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))
            self._nv = pynvml
            self.source = "nvml"
        except Exception:
            self._index = device.index or 0
            self.source = "nvidia-smi"

    def _reasons(self):
        nv = self._nv
        for name in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            fn = getattr(nv, name, None)
            if fn is not None:
                try:
                    return int(fn(self._handle))
                except Exception:
                    continue
        return 0

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                sm = float(nv.nvmlDeviceGetClockInfo(self._handle, nv.NVML_CLOCK_SM))
                pw = nv.nvmlDeviceGetPowerUsage(self._handle) / 1000.0
                self.samples.append((time.perf_counter(), sm, pw, self._reasons()))
            except Exception:
                pass
            self._stop.wait(0.002)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
            return
        try:
            self._file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self._smi = subprocess.Popen(["nvidia-smi", "-i", str(self._index), "--query-gpu=" + self.SMI_FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=self._file, stderr=subprocess.DEVNULL)
        except Exception:
            self._smi = None

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        if self._smi is not None:
            self._smi.terminate()
            try:
                self._smi.wait(timeout=5)
            except Exception:
                self._smi.kill()
            self._file.flush()
            self._file.seek(0)
            now = time.perf_counter()
            for line in self._file:
                parts = [p.strip() for p in line.split(",")]
                try:
                    sm, mx, pw = float(parts[0]), float(parts[1]), float(parts[2])
                except (ValueError, IndexError):
                    continue
                bits = 0
                for bit, val in zip((0x8, 0x40, 0x20, 0x4), parts[3:7]):
                    if val.lower().startswith("active"):
                        bits |= bit
                self.max_mhz = mx
                self.samples.append((now, sm, pw, bits))   # no usable timestamps: whole-run samples
            self._file.close()
            os.unlink(self._file.name)

    def region(self, t0, t1):
        """Summary of the samples taken inside [t0, t1] (host clock)."""
        inside = [s for s in self.samples if t0 <= s[0] <= t1] if self.source == "nvml" else list(self.samples)
        note = None
        if not inside and self.samples:    # a region shorter than the sampling period: the nearest sample
            mid = 0.5 * (t0 + t1)
            inside = [min(self.samples, key=lambda s: abs(s[0] - mid))]
            note = "region shorter than the sampling period: nearest sample"
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "source": self.source}
        if inside:
            bits = 0
            for s in inside:
                bits |= s[3]
            out.update(sm_mhz=statistics.median(s[1] for s in inside), sm_mhz_min=min(s[1] for s in inside),
                       power_w_max=max(s[2] for s in inside), samples=len(inside) if note is None else 0,
                       reasons=[name for bit, name in self.REASONS if bits & bit])
        if note:
            out["note"] = note
        return out


# ------------------------------------------------------------------------------------ distributed helpers


def dist_setup(n_gpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:    # launched by torch.distributed.run, even with one rank: use the collective
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        os.environ.setdefault("RANK", "0")
        os.environ.setdefault("WORLD_SIZE", "1")
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


# ------------------------------------------------------------------------------------ oracle legs


def oracle_modes():
    import oracle
    return {"greedy": oracle.GREEDY, "stochastic": oracle.STOCHASTIC}


def run_oracle(w, mode, x_host, n_threads, n_keep):
    """The oracle as it stands on host copies of the inputs: (seconds, outputs, selected)."""
    import oracle
    t0 = time.perf_counter()
    o = oracle.score_windows(x_host["draft_logits"], x_host["target_logits"], x_host["draft_tokens"],
                             mode=oracle_modes()[mode], c=w.c, temperature=w.temperature,
                             uniforms=x_host["uniforms"], valid_len=x_host["valid_len"], n_threads=n_threads)
    sel = oracle.select_windows(o["score"], min(n_keep, len(o["score"])))
    return time.perf_counter() - t0, o, sel


def host_sample(w, chunks, device):
    x = W.generate(w, device, chunks=chunks)
    return {k: (None if v is None else v.cpu()) for k, v in x.items()}


def _outside(g, o):
    g = np.asarray(g, np.float64)
    o = np.asarray(o, np.float64)
    same_inf = np.isinf(g) & np.isinf(o) & (np.sign(g) == np.sign(o))
    with np.errstate(invalid="ignore"):
        ok = np.abs(g - o) <= ATOL + RTOL * np.abs(o)
    return ~(ok | same_inf)


def parity_counts(B, w, mode, x, out, ref, ref_sel, windows, keep_pct):
    """Counts of disagreements between the GPU outputs of the timed buffers and the oracle's outputs for the
    windows `windows` (a slice).  Integer results must agree exactly; stochastic flags may differ only inside
    the 1e-6 band around u = alpha (counted, and their windows left out of the accepted-length comparison);
    floats within 1e-6 + 1e-4 |oracle|; the selection is checked on the sample's own scores."""
    import oracle
    fields = ("target_argmax", "accept_flag", "accepted_len", "kl", "conf", "crit", "logp_tok", "logq_tok",
              "reward_speedup", "reward_dist", "reward", "delta", "score")
    g = {k: out[k][windows].detach().cpu().numpy() for k in fields}
    ints = int((g["target_argmax"] != ref["target_argmax"]).sum())
    differ = g["accept_flag"] != ref["accept_flag"]
    band = 0
    band_windows = np.zeros(differ.shape[0], bool)
    if mode == "greedy":
        ints += int(differ.sum())
    else:
        u = x["uniforms"][windows].detach().cpu().numpy().astype(np.float64)
        in_band = np.abs(ref["alpha"] - u) < BAND
        ints += int((differ & ~in_band).sum())
        band = int((differ & in_band).sum())
        band_windows = differ.any(axis=1)
    keep = ~band_windows
    ints += int((g["accepted_len"][keep] != ref["accepted_len"][keep]).sum())
    floats = 0
    for f in ("kl", "conf", "crit", "logp_tok", "logq_tok"):
        floats += int(_outside(g[f], ref[f]).sum())
    for f in ("reward_speedup", "delta", "score"):
        floats += int(_outside(g[f][keep], ref[f][keep]).sum())
    near_eps = np.abs(ref["delta"] - 0.5) <= ATOL + RTOL * 0.5        # reward_dist is a threshold on delta (eps = 0.5)
    k2 = keep & ~near_eps
    ints += int((g["reward_dist"][k2] != ref["reward_dist"][k2].astype(np.float32)).sum())
    floats += int(_outside(g["reward"][k2], ref["reward"][k2]).sum())
    # selection: (i) the library's selection against the oracle's on the identical float32 scores, bit-exact;
    # (ii) against the oracle's selection on its own float64 scores: only windows at the cut may differ
    ns = g["score"].shape[0]
    nk = (keep_pct * ns + 99) // 100
    sel = B.select_windows(out["score"][windows].contiguous(), nk)
    torch.cuda.synchronize()
    sel = sel.cpu().numpy()
    want = oracle.select_windows(g["score"].astype(np.float64), nk)
    ints += int((sel != want).sum())
    swaps = 0
    ref_sel = oracle.select_windows(ref["score"], nk)
    if 0 < nk < ns:
        cut = ref["score"][ref_sel[-1]]
        for i in set(sel.tolist()) ^ set(ref_sel.tolist()):
            if abs(ref["score"][i] - cut) <= 2 * (ATOL + RTOL * abs(cut)):
                swaps += 1
            else:
                ints += 1
    return {"windows_checked": int(ns), "int_mismatches": ints, "float_out_of_tol": floats, "band_flags": band,
            "near_cut_swaps": swaps}


# -------------------------------------------------------------------------------------- reference arm


def run_reference(args):
    """Times the float64 CPU oracle (as it stands) on the machine's host cores; rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = W.BY_NAME[args.workload]
    if args.windows:
        w = W.scaled(w, args.windows, name=w.name)
    if args.logits:
        w = dataclasses.replace(w, dtype=args.logits)
    mode = args.mode or w.modes[-1]
    cores = os.cpu_count() or 1
    gen_dev = torch.device("cuda:0") if torch.cuda.is_available() else torch.device("cpu")
    n_chunks = (w.N + W.CHUNK - 1) // W.CHUNK
    samples = [host_sample(w, [i % n_chunks], gen_dev) for i in range(min(4, n_chunks))]
    times = []
    for i in range(args.warmup + args.steps):
        xs = samples[i % len(samples)]
        dt, _, _ = run_oracle(w, mode, xs, cores, (w.keep_pct * xs["draft_tokens"].shape[0] + 99) // 100)
        if i >= args.warmup:
            times.append(dt)
    windows = samples[0]["draft_tokens"].shape[0]
    total = sum(times)
    value = windows * len(times) / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "windows/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, mode),
        "cpu_baseline": {"value": value, "unit": "windows/s", "cores": cores, "kind": "oracle",
                         "sample": "sampled: each step scores one %d-window chunk of %s (not all N windows), float64 C "
                                   "oracle with pthreads" % (windows, w.name)},
        "e2e": {"value": value, "unit": "windows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# -------------------------------------------------------------------------------------- ppow arm


def _group_is_up():
    import torch.distributed as dist
    return dist.is_available() and dist.is_initialized()


class Run:
    """One workload resident on the device, with the calls of a step prepared."""

    def __init__(self, B, S, w, mode, dev, rank=0, world=1, train=False):
        self.B, self.S, self.w, self.mode, self.dev, self.world, self.train = B, S, w, mode, dev, world, train
        n_chunks = (w.N + W.CHUNK - 1) // W.CHUNK
        # weak scaling: rank r scores windows [r*N, (r+1)*N) of a world*N-window instance of the workload
        wg = W.scaled(w, w.N * world, name=w.name)
        self.x = x = W.generate(wg, dev, chunks=range(rank * n_chunks, (rank + 1) * n_chunks))
        N, K, V = w.N, w.K, w.V
        self.n_total, self.n_keep = N * world, wg.n_keep
        bmode = B.PPOW_GREEDY if mode == "greedy" else B.PPOW_STOCHASTIC
        self.params = B.make_params(N, K, V, {"f32": B.PPOW_F32, "bf16": B.PPOW_BF16, "f16": B.PPOW_F16}[w.dtype],
                                    bmode, w.c, w.temperature)
        self.out = B.alloc_outputs(N, K, dev)
        if train:
            self.out.update(B.alloc_train_outputs(N, K, dev))
            self.advantage = torch.empty((N,), dtype=torch.float32, device=dev)
            self.exp_accept = torch.empty((N, K), dtype=torch.float32, device=dev)
            self.ref_logp = torch.empty((N,), dtype=torch.float32, device=dev)
            self.row_logp = torch.empty((N, K), dtype=torch.float32, device=dev)
            self.group = 8 if N % 8 == 0 else 1
        self.ws = B.alloc_workspace(B.ppow_score_workspace_bytes(self.params), dev)
        self.selected = torch.empty((self.n_keep,), dtype=torch.int32, device=dev)
        self.sel_ws = B.alloc_workspace(B.ppow_select_workspace_bytes(self.n_total), dev)
        self.stream = torch.cuda.current_stream()
        self.score_call = B.ScoreCall(self.params, x["draft_logits"], x["target_logits"], x["draft_tokens"],
                                      x["uniforms"], x["valid_len"], None, self.out, self.ws)
        self.dtype_code = self.params.dtype
        self.gather = world > 1 or _group_is_up()    # one rank under torch.distributed.run still gathers (same values)
        self.select_call = None if self.gather else B.SelectCall(self.out["score"], self.n_keep, self.selected, None, self.sel_ws)
        self.acc_events, self.ref_events = [], []
        self.valid_rows = int(x["valid_len"].sum().item()) if x["valid_len"] is not None else N * K
        self.esize = 4 if w.dtype == "f32" else 2
        self.algo_bytes = 2 * self.valid_rows * V * self.esize    # both logit tensors, read once per launch of the row kernel
        self.launches_per_step = B.ppow_score_kernel_launches(self.params) + 1 + (4 if train else 0)

    def set_mode(self, mode):
        """Score the same buffers under the other acceptance test."""
        B, w, x = self.B, self.w, self.x
        self.mode = mode
        self.params = B.make_params(w.N, w.K, w.V, self.dtype_code, B.PPOW_GREEDY if mode == "greedy" else B.PPOW_STOCHASTIC,
                                    w.c, w.temperature)
        self.score_call = B.ScoreCall(self.params, x["draft_logits"], x["target_logits"], x["draft_tokens"],
                                      x["uniforms"], x["valid_len"], None, self.out, self.ws)

    def step(self, ev0=None, ev1=None):
        B, x, out, stream = self.B, self.x, self.out, self.stream
        self.score_call.launch(stream, ev0, ev1)
        if self.train:
            B.ppow_group_advantage(out["reward"], self.group, 1e-6, self.advantage, stream)
            ea = eb = None
            if ev0 is not None:
                ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                ea.record(stream)
            B.ppow_expected_acceptance(self.params, x["draft_logits"], x["target_logits"], x["valid_len"], out["lse_p"],
                                       out["lse_q"], self.exp_accept, stream)
            if ea is not None:
                eb.record(stream)
                self.acc_events.append((ea, eb))
            # the target's logits stand in for the logits along its reference window (same shape and type)
            B.ppow_reference_logprob(self.params, x["target_logits"], x["valid_len"], self.row_logp, self.ref_logp, stream)
            if ea is not None:
                ec = torch.cuda.Event(enable_timing=True)
                ec.record(stream)
                self.ref_events.append((eb, ec))
        if self.gather:
            scores = self.S.gather_scores(out["score"], self.n_total)    # the one exchange step
            B.ppow_select_windows(scores, self.n_keep, self.selected, None, self.sel_ws, stream)
        else:
            self.select_call.launch(stream)

    def measure(self, steps, warmup, trace=True):
        """`steps` timed steps after `warmup` untimed ones.  Returns device times and the host timestamps that
        bracket the timed region (for the clock samples).  `trace`: also time the row kernel of every step alone
        (two more event records per step, which shows on steps of a few microseconds)."""
        for _ in range(warmup):
            self.step()
        torch.cuda.synchronize()
        ev_pairs = [((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) if trace else (None, None))
                    for _ in range(steps)]
        for a, b in ev_pairs:
            if trace:
                a.record(), b.record()                  # create the CUDA events before the timed region
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier(self.world)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        start.record()
        for a, b in ev_pairs:
            self.step(a, b)
        stop.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        barrier(self.world)
        elapsed_ms = max_over_ranks(start.elapsed_time(stop), self.world, self.dev)
        reduce_ms = [a.elapsed_time(b) for a, b in ev_pairs] if trace else [float("nan")]
        reduce_avg_ms = max_over_ranks(sum(reduce_ms) / len(reduce_ms), self.world, self.dev)
        return {"elapsed_ms": elapsed_ms, "step_ms": elapsed_ms / steps, "kernel_ms": reduce_avg_ms, "t0": t0, "t1": t1,
                "steps": steps}

    def plain_kernel_ms(self, steps):
        """Row kernel of the plain scoring pass (no training-side outputs) on this run's buffers, by events."""
        B, x = self.B, self.x
        out = B.alloc_outputs(self.w.N, self.w.K, self.dev)
        call = B.ScoreCall(self.params, x["draft_logits"], x["target_logits"], x["draft_tokens"], x["uniforms"],
                           x["valid_len"], None, out, self.ws)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in pairs:
            a.record(), b.record()
        for _ in range(3):
            call.launch(self.stream)
        torch.cuda.synchronize()
        for a, b in pairs:
            call.launch(self.stream, a, b)
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in pairs) / steps

    def free(self):
        for name in ("x", "out", "ws", "score_call", "select_call", "sel_ws", "selected"):
            setattr(self, name, None)
        torch.cuda.empty_cache()


def read_only_probe(B, run, iters=10):
    """GB/s of a read-only streaming pass (16-byte loads, XOR fold) over the run's two logit tensors."""
    chk = torch.zeros((1,), dtype=torch.int32, device=run.dev)
    a, b = run.x["target_logits"], run.x["draft_logits"]
    nbytes = (a.numel() + b.numel()) * a.element_size()
    for _ in range(2):
        B.ppow_stream_read_probe(a, chk), B.ppow_stream_read_probe(b, chk)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        B.ppow_stream_read_probe(a, chk), B.ppow_stream_read_probe(b, chk)
    e1.record()
    torch.cuda.synchronize()
    return nbytes * iters / (e0.elapsed_time(e1) * 1e-3) / 1e9, nbytes


def oracle_leg(B, run, n_windows, cores):
    """Oracle on the first n_windows of the run's buffers: timing (cpu_baseline) and parity counts."""
    w, x = run.w, run.x
    idx = slice(0, min(w.N, n_windows))
    xs = {k: (None if v is None else v[idx].cpu()) for k, v in x.items()}
    nw = xs["draft_tokens"].shape[0]
    dt, ref, ref_sel = run_oracle(w, run.mode, xs, cores, (w.keep_pct * nw + 99) // 100)
    parity = parity_counts(B, w, run.mode, x, run.out, ref, ref_sel, idx, w.keep_pct)
    return dt, nw, parity


def workload_entry(B, run, steps, sampler, peak, cores, with_oracle=True):
    """One entry of "workloads": throughput of the row kernel and of the step, clocks inside the timed region,
    and the parity counts of a small sample against the oracle."""
    w, mode = run.w, run.mode
    m = run.measure(steps, 3, trace=False)                       # the step as a caller runs it
    m["kernel_ms"] = run.measure(min(steps, 200), 0)["kernel_ms"]    # and the row kernel alone
    flags = B.ppow_read_error_flags(run.ws)
    entry = {"workload": w.name, "mode": mode, "N": w.N, "K": w.K, "V": w.V, "logits": w.dtype, "steps": steps,
             "ms_per_step": m["step_ms"], "windows_per_s": w.N / (m["step_ms"] * 1e-3),
             "kernel_ms": m["kernel_ms"], "valid_row_bytes": run.algo_bytes,
             "logit_gbs": run.algo_bytes / (m["kernel_ms"] * 1e-3) / 1e9,
             "frac": run.algo_bytes / (m["kernel_ms"] * 1e-3) / 1e9 / peak,
             "frac_of_nominal_8TBs": run.algo_bytes / (m["kernel_ms"] * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
             "hbm_figure": run.algo_bytes > 4e8, "clocks": sampler.region(m["t0"], m["t1"]), "error_flags": flags}
    entry["parity"] = entry["oracle"] = None
    if with_oracle:
        dt, nw, entry["parity"] = oracle_leg(B, run, PARITY_SAMPLE_WINDOWS, cores)
        entry["oracle"] = {"windows_per_s": nw / dt, "cores": cores, "sample": "first %d windows" % nw}
    return entry


def training_figures(run, m):
    """Throughput of the training-side streaming kernels of a --train run (row kernel with the KL(Q||P) sum,
    expected-acceptance pass over both tensors, reference-window log-probability pass over one)."""
    acc_ms = sum(a.elapsed_time(b) for a, b in run.acc_events) / len(run.acc_events)
    ref_ms = sum(a.elapsed_time(b) for a, b in run.ref_events) / len(run.ref_events)
    return {"logits": run.w.dtype, "kl_rev_in_scoring_pass": True, "group_size": run.group,
            "row_reduce_with_kl_rev_ms": m["kernel_ms"], "row_reduce_with_kl_rev_gbs": run.algo_bytes / (m["kernel_ms"] * 1e-3) / 1e9,
            "expected_acceptance_ms": acc_ms, "expected_acceptance_gbs": run.algo_bytes / (acc_ms * 1e-3) / 1e9,
            "reference_logprob_ms": ref_ms, "reference_logprob_gbs": 0.5 * run.algo_bytes / (ref_ms * 1e-3) / 1e9}


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
        w = dataclasses.replace(w, dtype=args.logits)
    mode = args.mode or w.modes[-1]
    solo = world == 1
    cores = os.cpu_count() or 1
    peak, peak_kind = measured_peak()

    run = Run(B, S, w, mode, dev, rank, world, train=args.train)
    N, K, V = w.N, w.K, w.V
    sampler = ClockSampler(dev)
    if rank == 0:
        sampler.start()
        time.sleep(0.05)

    # ---- the K timed steps (value), after W >= 3 warm-up steps
    warmup = max(args.warmup, 3)
    m = run.measure(args.steps, warmup)
    flags = B.ppow_read_error_flags(run.ws)
    clocks = sampler.region(m["t0"], m["t1"]) if rank == 0 else None
    achieved = run.algo_bytes / (m["kernel_ms"] * 1e-3) / 1e9
    training = training_figures(run, m) if args.train else None

    # ---- the same step for at least SUSTAINED_SECONDS: the regime under the board's power limit
    sustained = None
    if solo and not args.no_sustained and not args.train:
        n_long = max(args.steps, int(math.ceil(SUSTAINED_SECONDS / (m["step_ms"] * 1e-3))))
        ms = run.measure(n_long, 0)
        cs = sampler.region(ms["t0"], ms["t1"])
        got = run.algo_bytes / (ms["kernel_ms"] * 1e-3) / 1e9
        sustained = {"seconds": ms["elapsed_ms"] * 1e-3, "steps": n_long, "ms_per_step": ms["step_ms"],
                     "windows_per_s": N / (ms["step_ms"] * 1e-3), "kernel_ms": ms["kernel_ms"], "achieved": got,
                     "frac": got / peak, "clocks": cs,
                     "kernel_ms_x_sm_mhz": (ms["kernel_ms"] * cs["sm_mhz"]) if cs.get("sm_mhz") else None}

    # ---- a read-only streaming pass over the same buffers, from the library
    read_only = None
    if solo and not args.no_probe:
        gbs, nbytes = read_only_probe(B, run)
        read_only = {"gbs": gbs, "bytes_per_pass": nbytes, "frac_of_read_only": achieved / gbs,
                     "how": "ppow_stream_read_probe over the two logit tensors of this run, 10 passes, CUDA events"}

    # ---- the oracle, as it stands, on this machine's host cores, and its outputs against the GPU's (rank 0, N = 1 only)
    cpu_baseline = parity = None
    if rank == 0 and solo and not args.no_cpu_baseline and not args.train:
        import oracle
        oracle.build()
        n_sample = min(N, 16 * W.CHUNK)         # ~25 core-seconds of oracle work on the headline workload
        dt, nw, parity = oracle_leg(B, run, n_sample, cores)
        cpu_baseline = {"value": nw / dt, "unit": "windows/s", "cores": cores, "kind": "oracle",
                        "sample": "sampled: first %d of %d windows of %s, float64 C oracle with pthreads, %.1f s wall"
                                  % (nw, N, w.name, dt)}

    # ---- end to end through the host-buffer entry point: pinned host inputs -> results on the host
    e2e = None
    if not args.no_e2e:
        x, out = run.x, run.out
        host = {k: (None if v is None else v.cpu().pin_memory()) for k, v in x.items()}
        out_host = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in out.items()}
        sel_host = torch.empty((w.n_keep,), dtype=torch.int32).pin_memory()
        scratch = B.alloc_workspace(B.ppow_host_scratch_bytes(run.params, N), dev)

        def e2e_step():
            B.ppow_score_and_select_host(run.params, host["draft_logits"], host["target_logits"], host["draft_tokens"],
                                         host["uniforms"], host["valid_len"], None, out_host, w.n_keep, sel_host,
                                         None, scratch, run.stream)
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
        e2e = {"value": run.n_total * e2e_steps / e2e_s, "unit": "windows/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": 1e3 * e2e_s / e2e_steps,
               "note": "ppow_score_and_select_host: pinned host logits copied to the device inside the timed region"}
        # the same call with scratch for an eighth of the windows at a time (eight staged chunks on the one stream)
        if solo and N >= 64:
            small = B.alloc_workspace(B.ppow_host_scratch_bytes(run.params, N // 8), dev)
            scratch = small
            e2e_step()
            t0 = time.perf_counter()
            for _ in range(3):
                e2e_step()
            dt = (time.perf_counter() - t0) / 3
            e2e["chunked"] = {"chunk_windows": N // 8, "scratch_bytes": int(small.numel()), "value": run.n_total / dt,
                              "ms_per_step": 1e3 * dt}
            del small
        del host, out_host, scratch

    # ---- one entry per other workload (generated, timed, checked and freed one at a time)
    workloads = None
    run_gather = run.gather
    launches_per_step, algo_bytes, n_total, n_keep = run.launches_per_step, run.algo_bytes, run.n_total, run.n_keep
    selected_checksum = int(torch.sum(run.selected.to(torch.int64) * torch.arange(1, n_keep + 1, device=dev)).item()) if n_keep else 0
    if rank == 0 and solo and not args.no_workloads and args.workload == "llama3_like" and not (args.windows or args.logits or args.train):
        run.free()
        workloads = []
        plan = {"tiny": 2000, "vicuna_like": 300, "qwen_like": 40, "heavy_tail": 20}
        for ow in W.WORKLOADS:
            if ow.name == w.name:
                continue
            other = Run(B, S, ow, ow.modes[0], dev)
            for om in ow.modes:                 # heavy_tail: the same buffers under both acceptance tests
                other.set_mode(om)
                workloads.append(workload_entry(B, other, plan[ow.name], sampler, peak, cores,
                                                with_oracle=not args.no_cpu_baseline))
            other.free()
            del other
        # the training-side streaming kernels on the headline shape in each storage type
        training = []
        for lg in ("bf16", "f16", "f32"):
            tr = Run(B, S, dataclasses.replace(w, dtype=lg), mode, dev, train=True)
            mt = tr.measure(20, 3)
            fig = training_figures(tr, mt)
            fig["clocks"] = sampler.region(mt["t0"], mt["t1"])
            plain_ms = tr.plain_kernel_ms(20)
            fig["row_reduce_ms"], fig["row_reduce_gbs"] = plain_ms, tr.algo_bytes / (plain_ms * 1e-3) / 1e9
            training.append(fig)
            tr.free()
            del tr

    if rank == 0:
        sampler.stop()
    if rank != 0:
        return
    value = n_total / (m["step_ms"] * 1e-3)
    per_window = NCU_TRAFFIC_BYTES_PER_WINDOW.get(w.name)
    line = {
        "metric": METRIC, "value": value, "unit": "windows/s", "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": m["step_ms"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "storage_dtype": w.dtype, "data": "synthetic",
        "config": config_of(w, mode), "n_keep_global": n_keep, "selected_checksum": selected_checksum,
        "score_exchange": "all_gather over the process group" if run_gather else "none (no process group)",
        "logit_gbs": world * algo_bytes / (m["step_ms"] * 1e-3) / 1e9,
        "roofline": {"bound": "hbm", "kernel": "row_reduce", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": "of " + peak_kind, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "traffic": (per_window * N if per_window and w.dtype == "bf16" and not args.train else None),
                     "traffic_source": "ncu dram__bytes_read+write on a 256-window capture (1.0056 x algorithmic), scaled "
                                       "by windows (null: other workload, storage type or kernel instance)",
                     "algorithmic_bytes_per_launch": algo_bytes, "kernel_ms": m["kernel_ms"],
                     "read_only_peak": read_only, "sustained": sustained},
        "parity": parity, "workloads": workloads, "training": training,
        "e2e": e2e, "cpu_baseline": cpu_baseline, "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
        "error_flags": flags,
    }
    print(json.dumps(line))
    bad = [p for p in ([parity] + [e["parity"] for e in (workloads or [])]) if p and (p["int_mismatches"] or p["float_out_of_tol"])]
    if bad:
        sys.stderr.write("parity check failed: %r\n" % bad)
        sys.exit(3)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ppow(args)
    if _group_is_up():
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
