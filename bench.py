#!/usr/bin/env python
"""Benchmark of the decode-attention hot path over a head-mixed KV cache.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama8b|qwen7b|cot|tiny]
                    [--frac F] [--context C] [--batch B] [--layers L] [--impl ours|reference]
                    [--no-configs] [--loop] [--sweep] [--sweep-table FILE]

One "step" = for every layer: append one token, then decode attention, over a cache that already
holds `context` tokens.  Prints ONE JSON line (rank 0).  Inputs are synthetic, seeded, bf16 N(0,1);
head classes come from a seeded global selection (see synth/).

  value      tokens/s = N * batch / (median time of one of K consecutive steps, device-timed, max over
             ranks), inputs resident in HBM (rlkv_step); the mean over the whole timed region is kept
             beside it (ms_per_step_mean)
  roofline   the decode kernel: algorithmic K/V bytes per launch / mean launch duration over the timed
             region; `isolated` = every rlkv_decode_attention launch of K more steps timed alone;
             `read_only_stream` = this GPU's read-only HBM bandwidth measured in the same run with the
             producer's copy mechanism and no consumer (rlkv_debug_read_bandwidth)
  e2e        the same K steps through rlkv_step_host: pinned host inputs copied in and the result
             copied out inside the timed region
  configs    (N = 1) the other workloads of the headline metric, each with its bytes, GB/s, clocks and
             the cost-model ratio beside the measured one: the Qwen-like shape at 60 % and at 0 %, the
             Llama-like shape at 0/20/40/60/80 % of the KV heads compressed, and the long decode loop
             (4096-token prompt, then every one of 28672 steps, fresh inputs per step)
  cpu_baseline  the CPU oracle on a bounded sample (rank 0, N = 1 only), scaled by bytes
  mixed_attention, paged_cache   side measurements at N = 1 (not part of `value`)

--loop runs only the long decode loop (on --workload cot); --sweep prints one JSON line per cell of
the compression x context x batch grid instead of the bench line, and --sweep-table FILE turns such
lines into a markdown table.

With N > 1 (torchrun) every rank runs the same workload on its own GPU: the path shards by batch
rows / replicas with no exchange step, so there is no collective on the data path (weak scaling).
--impl reference times the CPU oracle alone on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import synth

METRIC = "decode-attn tokens/s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
SWEEP_FRACS = (0.0, 0.2, 0.4, 0.6, 0.8)
SWEEP_CONTEXTS = (2048, 8192, 32768, 65536)
SWEEP_BATCHES = (1, 8, 32, 64)
SWEEP_CACHE_BYTES = 100 * 2**30        # most K/V bytes a sweep cell holds on the device
LOOP_STEPS = 28672                     # generated steps of the long decode loop (prompt 4096 -> n = 32768)
LOOP_BLOCK = 64                        # steps between two timing events of the loop


# ------------------------------------------------------------------------------------------------
def parse_args(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=20)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", choices=["ours", "reference"], default="ours")
    p.add_argument("--workload", default="llama8b", choices=sorted(synth.WORKLOADS))
    p.add_argument("--frac", type=float, default=None, help="override the fraction of compressed KV heads")
    p.add_argument("--context", type=int, default=None)
    p.add_argument("--batch", type=int, default=None)
    p.add_argument("--layers", type=int, default=None)
    p.add_argument("--ctas-per-sm", type=int, default=0)
    p.add_argument("--stages", type=int, default=0)
    p.add_argument("--groups", type=int, default=0, help="consumer warp groups of the decode kernel")
    p.add_argument("--item-tiles", type=int, default=0, help="smallest work item of the decode kernel, in 64-row tiles")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--no-mixed", action="store_true", help="skip the mixed-attention (Eq. 1) side measurement")
    p.add_argument("--no-paged", action="store_true", help="skip the paged, ragged cache side measurement")
    p.add_argument("--no-configs", action="store_true", help="skip the other workloads of the metric (`configs`)")
    p.add_argument("--loop", action="store_true", help="run only the long decode loop on the chosen workload")
    p.add_argument("--loop-steps", type=int, default=LOOP_STEPS)
    p.add_argument("--sweep", action="store_true", help="print one JSON line per cell of the compression sweep")
    p.add_argument("--sweep-contexts", type=int, nargs="*", default=list(SWEEP_CONTEXTS))
    p.add_argument("--sweep-batches", type=int, nargs="*", default=list(SWEEP_BATCHES))
    p.add_argument("--sweep-fracs", type=float, nargs="*", default=list(SWEEP_FRACS))
    p.add_argument("--sweep-table", default=None, help="print the markdown table of a file of --sweep lines and exit")
    return p.parse_args(argv)


def pick_workload(args) -> synth.Workload:
    w = synth.WORKLOADS[args.workload]
    kw = {}
    if args.frac is not None:
        kw["frac_compressed"] = args.frac
    if args.context is not None:
        kw["context"] = args.context
    if args.batch is not None:
        kw["batch"] = args.batch
    if args.layers is not None:
        kw["layers"] = args.layers
    return w.with_(**kw) if kw else w


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier pool measurement)"


def profiled_traffic_ratio():
    """DRAM bytes / algorithmic bytes of the decode kernel from the committed ncu summary, or None when
    the kernel source has changed since the counters were taken."""
    import hashlib
    import re
    prof = os.path.join(ROOT, "profiles", "decode_kernel_step_llama8b_4layers.md")
    csrc = os.path.join(ROOT, "paper_2510_08525_b200", "csrc")
    try:
        text = open(prof).read()
        h = hashlib.sha256()
        for name in ("decode_kernel.cu", "rlkv_internal.cuh"):
            h.update(open(os.path.join(csrc, name), "rb").read())
        want = re.search(r"kernel_source_sha256_16=([0-9a-f]+)", text).group(1)
        if h.hexdigest()[:16] != want:
            return None
        return float(re.search(r"traffic_ratio=([0-9.]+)", text).group(1))
    except Exception:
        return None


def max_over_ranks(value: float, device=None) -> float:
    """MAX of a per-rank scalar over the process group (identity without a group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while a timed region runs: through NVML
    every 2 ms where the Python bindings are there (read-only queries), else through nvidia-smi."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.gpu, self.rows, self.proc, self.thread, self.stop, self.how = gpu_index, [], None, None, False, None

    def wait_first_sample(self, timeout=3.0):
        t0 = time.perf_counter()
        while self.thread and not self.rows and time.perf_counter() - t0 < timeout:
            time.sleep(0.01)

    def mark(self):
        """Index of the next sample: samples from here on belong to what follows."""
        return len(self.rows)

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        try:
            uuid = torch.cuda.get_device_properties(self.gpu).uuid
            return pynvml, pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
        except Exception:
            return pynvml, pynvml.nvmlDeviceGetHandleByIndex(self.gpu)

    def __enter__(self):
        try:
            nv, h = self._nvml_handle()
            nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
            mx = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            bits = [(nv.nvmlClocksEventReasonHwSlowdown, 0), (nv.nvmlClocksEventReasonHwThermalSlowdown, 1),
                    (nv.nvmlClocksEventReasonSwThermalSlowdown, 2), (nv.nvmlClocksEventReasonSwPowerCap, 3)]

            def loop():
                while not self.stop:
                    try:
                        sm = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                        reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                        row = [str(sm), str(mx), ""] + ["Active" if reasons & bit else "Not Active" for bit, _ in bits]
                        self.rows.append(row)
                    except Exception:
                        pass
                    time.sleep(0.002)
            self.how = "nvml, every 2 ms"
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            return self
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.how = "nvidia-smi -lms 20"
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) == 7:
                self.rows.append(parts)

    def __exit__(self, *exc):
        self.stop = True
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread:
            self.thread.join(timeout=5)

    def summary(self, start=0, end=None):
        sm, mx, reasons = [], [], set()
        for r in self.rows[start:end]:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, r[3:]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "how": self.how}


# ------------------------------------------------------------------------------------------------
def workload_bytes(w: synth.Workload, mask: np.ndarray, n: int) -> int:
    """K/V bytes one decode step over all layers must read at length n (integer cost model)."""
    n_full = int(mask.sum())
    n_comp = mask.size - n_full
    rows = n_full * n + n_comp * min(n, w.sink + w.window)
    return w.batch * rows * 2 * w.head_dim * 2


def cost_model_ratio(w: synth.Workload, mask: np.ndarray, n: int) -> float:
    """(1 - s') + s' * min(n, sink + window) / n with s' the realised fraction of compressed heads:
    the paper's cost model (Section 4.3), which is also bytes(s') / bytes(0) exactly."""
    s = float((mask == 0).sum()) / mask.size
    return (1.0 - s) + s * min(n, w.sink + w.window) / n


def host_description():
    model = "unknown"
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                model = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    from oracle import rlkv_oracle
    try:
        cc = subprocess.run([rlkv_oracle.CC, "--version"], capture_output=True, text=True).stdout.splitlines()[0]
    except Exception:
        cc = rlkv_oracle.CC
    return {"cpu_model": model, "logical_cpus": os.cpu_count(), "compiler": cc, "flags": " ".join(rlkv_oracle.CFLAGS)}


def build_oracle_sample(w: synth.Workload, mask: np.ndarray, gen_device, target_bytes=200e6):
    from oracle.rlkv_oracle import Oracle
    n = w.context + 1
    layer_mask = mask[:w.kv_heads]
    per_row = workload_bytes(w.with_(batch=1, layers=1), layer_mask, n)
    sb = int(max(1, min(w.batch, target_bytes // max(per_row, 1))))
    oracle = Oracle(1, w.kv_heads, w.q_heads, w.head_dim, sb, n, layer_mask, w.sink, w.window)
    chunk = max(1, (1 << 23) // (w.batch * w.kv_heads * w.head_dim))
    for t0 in range(0, w.context, chunk):
        t1 = min(w.context, t0 + chunk)
        k = synth.rows(w.seed, synth.STREAM_K, 0, t0, t1, w.batch, w.kv_heads, w.head_dim, gen_device)[:, :sb].cpu()
        v = synth.rows(w.seed, synth.STREAM_V, 0, t0, t1, w.batch, w.kv_heads, w.head_dim, gen_device)[:, :sb].cpu()
        for t in range(t1 - t0):
            oracle.append(0, k[t].contiguous(), v[t].contiguous())
    t = w.context
    k1 = synth.rows(w.seed, synth.STREAM_K, 0, t, t + 1, w.batch, w.kv_heads, w.head_dim)[0, :sb].contiguous()
    v1 = synth.rows(w.seed, synth.STREAM_V, 0, t, t + 1, w.batch, w.kv_heads, w.head_dim)[0, :sb].contiguous()
    q = synth.rows(w.seed, synth.STREAM_Q, 0, t, t + 1, w.batch, w.q_heads, w.head_dim)[0, :sb].contiguous()
    sample_bytes = workload_bytes(w.with_(batch=sb, layers=1), layer_mask, n)
    desc = f"layer 0, batch rows 0..{sb - 1}, all {w.kv_heads} KV heads, n={n}: {sample_bytes / 1e6:.1f} MB of K/V"
    return oracle, (k1, v1, q), sample_bytes, desc


def time_oracle(oracle, step_in, threads: int, warmup: int, steps: int, min_seconds: float = 0.0):
    """Median seconds of one oracle decode over the sample: `warmup` untimed decodes, then at least
    `steps` timed ones and at least `min_seconds` of them (the append is done once, untimed:
    re-appending would grow the sample).  Both the cpu_baseline leg and --impl reference use this."""
    k1, v1, q = step_in
    oracle.set_threads(threads)
    if oracle.length(0) == oracle.max_len - 1:
        oracle.append(0, k1, v1)
    for _ in range(warmup):
        oracle.decode(0, q)
    times, t_all = [], time.perf_counter()
    while len(times) < steps or time.perf_counter() - t_all < min_seconds:
        t0 = time.perf_counter()
        oracle.decode(0, q)
        times.append(time.perf_counter() - t0)
    return statistics.median(times), len(times)


# ------------------------------------------------------------------------------------------------
def run_reference(args, w, mask):
    """--impl reference: the CPU oracle as it stands on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle.rlkv_oracle import max_threads
    gen_dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    oracle, step_in, sample_bytes, desc = build_oracle_sample(w, mask, gen_dev)
    threads = max_threads()
    per_sample, reps = time_oracle(oracle, step_in, threads, args.warmup, args.steps)
    total_bytes = workload_bytes(w, mask, w.context + 1)
    ms_per_step = per_sample * total_bytes / sample_bytes * 1e3
    value = w.batch / (ms_per_step / 1e3)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(w, mask),
        "note": "CPU oracle; each step = one decode over the sample (median of the timed decodes), scaled to the "
                "whole workload by K/V bytes",
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{desc}; median of {reps} decodes, scaled to the step by K/V bytes",
                         "host": host_description()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def config_dict(w, mask):
    n_comp = int((mask == 0).sum())
    return {"workload": w.name, "layers": w.layers, "q_heads": w.q_heads, "kv_heads": w.kv_heads,
            "head_dim": w.head_dim, "batch_per_gpu": w.batch, "context": w.context,
            "compressed_heads": f"{n_comp} of {mask.size}", "frac_compressed": w.frac_compressed,
            "sink": w.sink, "window": w.window, "seed": w.seed,
            "l2": "inputs larger than L2: every layer's K/V working set exceeds 126 MB and is read once per step"}


# ------------------------------------------------------------------------------------------------
def timed_steps(rl, harness, w, mask, dev, stream, K, W, clocks=None, tune=None, extra_tokens=0):
    """A cache of workload `w` filled to its context, then W untimed and K timed rlkv_step calls with
    one event between consecutive steps.  Returns (cache, steps_in, result); the caller closes the
    cache.  result: median and mean ms per step, the timed region's launches, bytes and clocks."""
    cache = harness.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, w.context + W + K + 8 + extra_tokens,
                          mask, w.sink, w.window, device=dev)
    if tune and any(tune):
        rl.rlkv_set_decode_config(cache.handle, *tune)
    harness.fill_cache(cache, w, w.context)
    steps_in = [harness.step_inputs(w, w.context + i, dev) for i in range(W + K)]
    out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    for i in range(W):
        rl.rlkv_step(cache.handle, *steps_in[i], out, stream)
    launches0 = rl.rlkv_launch_count(cache.handle)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    barrier(); torch.cuda.synchronize()
    mark0 = clocks.mark() if clocks else 0
    for i in range(K):
        ev[i].record(stream)
        rl.rlkv_step(cache.handle, *steps_in[W + i], out, stream)
    ev[K].record(stream)
    torch.cuda.synchronize()
    barrier()
    mark1 = clocks.mark() if clocks else 0
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(K)]
    region_ms = ev[0].elapsed_time(ev[K])
    n_mid = w.context + W + 1 + K // 2                    # the median step's length, near enough
    res = {"ms_per_step": statistics.median(per_step), "ms_per_step_mean": region_ms / K, "region_ms": region_ms,
           "ms_per_step_min": min(per_step), "ms_per_step_max": max(per_step),
           "launches": rl.rlkv_launch_count(cache.handle) - launches0,
           "kv_bytes_per_step": workload_bytes(w, mask, n_mid),
           "clocks": clocks.summary(mark0, mark1) if clocks else None,
           "out": out}
    return cache, steps_in, res


def config_entry(w, mask, res, peak):
    """What `configs` reports for one workload measured by timed_steps."""
    n = w.context + 1
    gbs = res["kv_bytes_per_step"] / (res["ms_per_step"] * 1e-3) / 1e9
    return {"workload": w.name, "batch": w.batch, "context": w.context, "layers": w.layers,
            "frac_compressed": w.frac_compressed, "compressed_heads": f"{int((mask == 0).sum())} of {mask.size}",
            "ms_per_step": res["ms_per_step"], "ms_per_step_mean": res["ms_per_step_mean"],
            "tokens_per_s": w.batch / (res["ms_per_step"] * 1e-3),
            "kv_bytes_per_step": res["kv_bytes_per_step"], "gbs": gbs, "frac_of_measured_copy": gbs / peak,
            "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS, "expected_ratio": cost_model_ratio(w, mask, n),
            "gpu_launches": res["launches"], "clocks": res["clocks"]}


def run_loop(rl, harness, w, mask, dev, stream, clocks, n_steps, peak):
    """The long decode loop: the prompt (w.context tokens) is prefilled, then every one of n_steps steps
    runs through rlkv_step with fresh seeded q, k, v generated on the device (synth/, not the library).
    Timed in blocks of LOOP_BLOCK steps (one event per block)."""
    n_end = w.context + n_steps
    cache = harness.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, n_end, mask, w.sink, w.window, device=dev)
    harness.fill_cache(cache, w, w.context)
    out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    gen_chunk = 256

    launches0 = rl.rlkv_launch_count(cache.handle)
    blocks = []                 # (first n of the block, steps, start event, end event)
    mark0 = clocks.mark() if clocks else 0
    wall0 = time.perf_counter()
    t = w.context
    while t < n_end:
        t1 = min(n_end, t + gen_chunk)
        k, v, q = harness.step_inputs_block(w, t, t1, dev)   # [steps][layers][batch][heads][head_dim]
        for b0 in range(0, t1 - t, LOOP_BLOCK):
            b1 = min(t1 - t, b0 + LOOP_BLOCK)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(b0, b1):
                rl.rlkv_step(cache.handle, k[i], v[i], q[i], out, stream)
            e1.record(stream)
            blocks.append((t + b0 + 1, b1 - b0, e0, e1))
        torch.cuda.synchronize()          # the chunk's inputs are freed only after its steps have run
        t = t1
    wall = time.perf_counter() - wall0
    mark1 = clocks.mark() if clocks else 0
    status = cache.status()
    if status != 0:
        raise SystemExit(f"a kernel of the decode loop reported status {status}: results are invalid")
    lengths = [rl.rlkv_length(cache.handle, l) for l in range(w.layers)]
    assert lengths == [n_end] * w.layers, lengths

    def block_stats(n_first, steps, e0, e1):
        ms = e0.elapsed_time(e1) / steps
        by = sum(workload_bytes(w, mask, n_first + i) for i in range(steps)) / steps
        return ms, by

    at = {}
    for target in (8192, 16384, 24576, 32768):
        hit = [b for b in blocks if b[0] <= target < b[0] + b[1]]
        if hit:
            ms, by = block_stats(*hit[-1])
            at[str(target)] = {"ms_per_step": ms, "kv_bytes_per_step": by, "gbs": by / (ms * 1e-3) / 1e9,
                               "frac_of_nominal_8000": by / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS}
    first = block_stats(*blocks[0])
    tail_steps, tail_ms, tail_bytes = 0, 0.0, 0.0
    for b in reversed(blocks):
        if tail_steps >= 1024:
            break
        ms, by = block_stats(*b)
        tail_steps += b[1]; tail_ms += ms * b[1]; tail_bytes += by * b[1]
    total_ms = sum(b[2].elapsed_time(b[3]) for b in blocks)
    total_bytes = sum(workload_bytes(w, mask, n) for n in range(w.context + 1, n_end + 1))
    res = {"workload": f"{w.name}: batch {w.batch}, prompt {w.context} prefilled, then {n_steps} steps to n = {n_end}, "
                       f"{int((mask == 0).sum())} of {mask.size} heads compressed, sink {w.sink} + window {w.window} "
                       f"(ring wrapped {(n_end - w.sink) // w.window} times), fresh seeded q/k/v every step",
           "steps": n_steps, "timed_in_blocks_of": LOOP_BLOCK,
           "first_block": {"n": blocks[0][0], "ms_per_step": first[0], "gbs": first[1] / (first[0] * 1e-3) / 1e9,
                           "frac_of_nominal_8000": first[1] / (first[0] * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
           "at_n": at,
           "steady_state_last_steps": tail_steps,
           "steady_state_ms_per_step": tail_ms / tail_steps,
           "steady_state_tokens_per_s": w.batch / (tail_ms / tail_steps * 1e-3),
           "steady_state_gbs": tail_bytes / tail_ms / 1e6,
           "steady_state_frac_of_measured_copy": tail_bytes / tail_ms / 1e6 / peak,
           "steady_state_frac_of_nominal_8000": tail_bytes / tail_ms / 1e6 / NOMINAL_HBM_GBS,
           "whole_loop_device_s": total_ms / 1e3, "whole_loop_gbs": total_bytes / total_ms / 1e6,
           "whole_loop_wall_s": wall, "expected_ratio_at_end": cost_model_ratio(w, mask, n_end),
           "gpu_launches": rl.rlkv_launch_count(cache.handle) - launches0,
           "checksum": float(out.double().abs().sum()),
           "clocks": clocks.summary(mark0, mark1) if clocks else None}
    cache.close()
    return res


def sweep_layers(w: synth.Workload) -> int:
    per_layer = w.kv_heads * w.batch * (w.context + 1) * 4 * w.head_dim      # at 0 % compressed
    return int(max(1, min(w.layers, SWEEP_CACHE_BYTES // per_layer)))


def run_sweep(args, rl, harness, dev, stream):
    """One JSON line per cell: compression x context x batch at the Llama-like shape.  The mask is
    drawn for all 32 layers and the first L' layers are held (as many as keep the cache under
    SWEEP_CACHE_BYTES at 0 %); times are per layer."""
    base = synth.WORKLOADS["llama8b"]
    K, W = max(args.steps, 3), max(args.warmup, 3)
    for ctx in args.sweep_contexts:
        for batch in args.sweep_batches:
            zero_us = None
            for frac in sorted(args.sweep_fracs):
                w32 = base.with_(context=ctx, batch=batch, frac_compressed=frac)
                lp = sweep_layers(w32)
                w = w32.with_(layers=lp)
                mask = synth.workload_mask(w32)[:lp * w.kv_heads]
                with ClockSampler(dev.index or 0) as clocks:
                    clocks.wait_first_sample(1.0)
                    cache, _, res = timed_steps(rl, harness, w, mask, dev, stream, K, W, clocks)
                    status = cache.status()
                    cache.close()
                if status != 0:
                    raise SystemExit(f"a kernel reported status {status}")
                by = res["kv_bytes_per_step"] / lp
                us = 1e3 * res["ms_per_step"] / lp
                if frac == 0.0:
                    zero_us = us
                n = ctx + 1
                s_real = float((mask == 0).sum()) / mask.size
                line = {"sweep": True, "context": ctx, "batch": batch, "frac": frac, "layers_held": lp,
                        "frac_realised": s_real, "us_per_layer": us, "kv_bytes_per_layer": by,
                        "gbs": by / (us * 1e-6) / 1e9, "frac_of_nominal_8000": by / (us * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
                        "expected_ratio": (1 - s_real) + s_real * min(n, base.sink + base.window) / n,
                        "measured_ratio": None if zero_us is None else us / zero_us,
                        "step_us": us * lp, "kv_bytes_per_step": by * lp,
                        # the whole step's K/V rows could partly stay in the 126 MB L2 from one step to the
                        # next / the step (one append launch, one attention launch) is set by latency
                        "l2_resident": by * lp < 252e6, "latency_bound": us * lp < 100.0,
                        "steps": K, "warmup": W, "clocks": res["clocks"]}
                print(json.dumps(line), flush=True)
                del res
                torch.cuda.empty_cache()


def sweep_table(path):
    """Markdown table of a file of --sweep lines: cells 'us per layer, TB/s (measured ratio / cost model)';
    † = the whole step reads less than twice the L2's size, ‡ = the whole step takes under 100 us."""
    cells = {}
    for line in open(path):
        line = line.strip()
        if not line.startswith("{"):
            continue
        d = json.loads(line)
        if d.get("sweep"):
            cells[(d["context"], d["batch"], d["frac"])] = d
    fracs = sorted({k[2] for k in cells})
    print("| context | batch | layers held | " + " | ".join(f"{int(round(100 * f))} %" for f in fracs) + " |")
    print("|---|---|---|" + "---|" * len(fracs))
    for ctx, batch in sorted({(k[0], k[1]) for k in cells}):
        row = []
        lp = None
        for f in fracs:
            d = cells.get((ctx, batch, f))
            if d is None:
                row.append("")
                continue
            lp = d["layers_held"]
            step_us, step_bytes = d["us_per_layer"] * lp, d["kv_bytes_per_layer"] * lp
            flag = ("†" if step_bytes < 252e6 else "") + ("‡" if step_us < 100.0 else "")
            ratio = "" if d["measured_ratio"] is None or f == 0 else f" ({d['measured_ratio']:.2f} / {d['expected_ratio']:.2f})"
            row.append(f"{d['us_per_layer']:.0f} µs, {d['gbs'] / 1e3:.2f} TB/s{flag}{ratio}")
        print(f"| {ctx} | {batch} | {lp} | " + " | ".join(row) + " |")


# ------------------------------------------------------------------------------------------------
def run_ours(args, w, mask):
    import torch.distributed as dist
    from paper_2510_08525_b200 import binding as rl
    from paper_2510_08525_b200 import harness

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: librlkv has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    stream = torch.cuda.current_stream()
    peak, peak_src = measured_peak_gbs()
    tune = (args.ctas_per_sm, args.stages, args.groups, args.item_tiles)

    if args.sweep:
        run_sweep(args, rl, harness, dev, stream)
        return
    if args.loop:
        with ClockSampler(local) as clocks:
            clocks.wait_first_sample()
            res = run_loop(rl, harness, w, mask, dev, stream, clocks, args.loop_steps, peak)
        print(json.dumps({"loop": res}), flush=True)
        return

    K, W = args.steps, args.warmup
    clocks = ClockSampler(local)
    clocks.__enter__()
    clocks.wait_first_sample()

    # ---- pass 1: device-resident steps (the headline value), one event between consecutive steps
    cache, steps_in, res = timed_steps(rl, harness, w, mask, dev, stream, K, W, clocks, tune, extra_tokens=2 * (K + W) + 24)
    out = res.pop("out")
    median_ms = max_over_ranks(res["ms_per_step"], dev)
    mean_ms = max_over_ranks(res["ms_per_step_mean"], dev)
    launches = res["launches"]
    value = world * w.batch / (median_ms / 1e3)
    main_clocks = res["clocks"]

    # ---- pass 2: per-launch CUDA events around every decode-attention launch
    more = [harness.step_inputs(w, w.context + W + K + i, dev) for i in range(W + K)]
    for i in range(W):
        rl.rlkv_step(cache.handle, *more[i], out, stream)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(K * w.layers)]
    bytes_launch = []
    torch.cuda.synchronize()
    for s in range(K):
        k, v, q = more[W + s]
        for l in range(w.layers):
            rl.rlkv_append(cache.handle, l, k[l], v[l], stream)
            a, b = ev[s * w.layers + l]
            a.record(stream)
            rl.rlkv_decode_attention(cache.handle, l, q[l], out[l], stream)
            b.record(stream)
            bytes_launch.append(rl.rlkv_step_bytes(cache.handle, l))
    torch.cuda.synchronize()
    durs = [a.elapsed_time(b) for a, b in ev]
    isolated = sum(bytes_launch) / (sum(durs) * 1e-3) / 1e9
    ratio = profiled_traffic_ratio()
    # this GPU's read-only stream, measured now: 2 GiB (larger than the L2) read with the producer's
    # copy mechanism and no consumer
    probe = torch.empty(2 << 30, dtype=torch.uint8, device=dev)
    probe_ms = rl.rlkv_debug_read_bandwidth(probe, probe.numel(), 6)
    read_only_gbs = probe.numel() / (probe_ms * 1e-3) / 1e9
    del probe
    # The decode launches of the timed region (pass 1): every step is one append launch and the step's
    # decode launches (one over all layers, or one per layer where the step had to fall back), between
    # the first and the last event on the launching stream.  Their average duration is taken as the
    # whole region divided by their number, which charges them the append launches too.
    n_launch = launches - K
    step_bytes = res["kv_bytes_per_step"]
    mean_launch_ms = mean_ms * K / n_launch
    bytes_per_launch = step_bytes * K / n_launch
    achieved = bytes_per_launch / (mean_launch_ms * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "rlkv::decode_kernel (whole-step mode)" if n_launch == K else "rlkv::decode_kernel",
        "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_source": peak_src, "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
        # ncu capture of a 4-layer cut of the workload (same kernel, same per-layer shape), scaled to
        # the mean launch of this run by the algorithmic bytes; null if the kernel has changed since
        "traffic": None if ratio is None else ratio * bytes_per_launch,
        "launches_timed": n_launch, "mean_launch_us": 1e3 * mean_launch_ms,
        "algorithmic_bytes_per_launch": bytes_per_launch,
        "how": "CUDA events on the launching stream around the timed region (K steps, each one append launch "
               "and its decode launches); duration = region / decode launches",
        "read_only_stream": {"gbs": read_only_gbs, "frac_of_it": achieved / read_only_gbs,
                             "how": "rlkv_debug_read_bandwidth: 2 GiB read by bulk copies into shared memory, "
                                    "no consumer, measured in this run"},
        "isolated": {"achieved": isolated, "frac": isolated / peak, "frac_of_nominal_8000": isolated / NOMINAL_HBM_GBS,
                     "mean_launch_us": 1e3 * sum(durs) / len(durs), "launches_timed": len(durs),
                     "how": "the per-layer call: every rlkv_decode_attention launch of K more steps timed alone "
                            "between two events"},
    }

    # ---- the per-layer calls as a model forward would issue them: before every layer a stand-in kernel
    # (a ~30 us device copy of the bench's own buffers) that consumes the layer before's output and
    # writes this layer's k, v, q at its end, then the append and the attention call.  Once with ordinary
    # launches (rlkv_append, rlkv_decode_attention), once with the overlapped calls and an overlapping
    # stand-in, once with rlkv_layer_step_overlapped (append and attention in one launch).  Attention time per layer = (chain - the same chain without the attention calls) / layers.
    per_layer = None
    if world == 1:
        kv_e, q_e = w.batch * w.kv_heads * w.head_dim, w.batch * w.q_heads * w.head_dim
        stage = torch.zeros(2 * kv_e + q_e, dtype=torch.bfloat16, device=dev)
        kb, vb, qb = stage[:kv_e], stage[kv_e:2 * kv_e], stage[2 * kv_e:]
        kk, vv, qq = more[0]
        srcs = [torch.cat([kk[l].reshape(-1), vv[l].reshape(-1), qq[l].reshape(-1)]) for l in range(w.layers)]
        work_src = torch.ones(96 << 20, dtype=torch.uint8, device=dev)
        work_dst = torch.empty_like(work_src)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 4

        def chain(overlap, attention):
            for l in range(w.layers):
                rl.rlkv_debug_standin(work_dst, work_src, work_src.numel(), out[l - 1] if l else None, stage, srcs[l],
                                      stage.numel() * 2, 1 if overlap else 0, stream)
                if attention and overlap == 2:
                    rl.rlkv_layer_step_overlapped(cache.handle, l, kb, vb, qb, out[l], stream)
                elif attention and overlap:
                    rl.rlkv_append_overlapped(cache.handle, l, kb, vb, stream)
                    rl.rlkv_decode_attention_overlapped(cache.handle, l, qb, out[l], stream)
                elif attention:
                    rl.rlkv_append(cache.handle, l, kb, vb, stream)
                    rl.rlkv_decode_attention(cache.handle, l, qb, out[l], stream)

        per_layer = {"workload": f"{w.name}: every layer = stand-in kernel (96 MiB device copy, writes the layer's k, v, q at "
                                 f"its end), append, attention; {reps} passes over the {w.layers} layers",
                     "kv_bytes_per_layer": step_bytes / w.layers}
        for name, overlap in (("ordinary", 0), ("overlapped", 1), ("overlapped_one_launch", 2)):
            t = {}
            for attention in (False, True):
                chain(overlap, attention)
                torch.cuda.synchronize()
                e0.record(stream)
                for _ in range(reps):
                    chain(overlap, attention)
                e1.record(stream)
                torch.cuda.synchronize()
                t[attention] = 1e3 * e0.elapsed_time(e1) / (reps * w.layers)
            us = t[True] - t[False]
            gbs = step_bytes / w.layers / (us * 1e-6) / 1e9
            per_layer[name] = {"standin_us": t[False], "chain_us_per_layer": t[True], "attention_us_per_layer": us,
                               "gbs": gbs, "frac_of_measured_copy": gbs / peak, "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS}
        del work_src, work_dst

    # ---- pass 3: end to end through rlkv_step_host (pinned host buffers, copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        host_in = [tuple(x.cpu().pin_memory() for x in s) for s in steps_in]
        out_host = torch.empty(out.shape, dtype=torch.float32).pin_memory()
        h2d = sum(x.numel() * x.element_size() for x in host_in[0])
        d2h = out_host.numel() * out_host.element_size()
        for i in range(W):
            rl.rlkv_step_host(cache.handle, *host_in[i], out_host, stream)
        barrier(); torch.cuda.synchronize()
        e0.record(stream)
        for i in range(W, W + K):
            rl.rlkv_step_host(cache.handle, *host_in[i], out_host, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), dev)
        e2e = {"value": world * w.batch * K / (e2e_ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / K,
               "checksum": float(out_host.double().abs().sum())}
        del host_in, out_host
    status = cache.status()
    if status != 0:
        raise SystemExit(f"a kernel reported status {status}: results are invalid")
    q0 = steps_in[0][2]
    kv0 = (steps_in[0][0], steps_in[0][1])
    cache.close()
    del steps_in, more
    torch.cuda.empty_cache()

    # ---- the other workloads of the metric (N = 1 only)
    configs = None
    if world == 1 and not args.no_configs and args.workload == "llama8b" and not any(
            x is not None for x in (args.frac, args.context, args.batch, args.layers)):
        configs = {}
        fr = []
        zero_ms = None
        for frac in SWEEP_FRACS:
            wf = w.with_(frac_compressed=frac)
            mf = synth.workload_mask(wf)
            if frac == w.frac_compressed:
                entry = config_entry(wf, mf, dict(res, ms_per_step=median_ms, ms_per_step_mean=mean_ms), peak)
            else:
                c2, _, r2 = timed_steps(rl, harness, wf, mf, dev, stream, K, W, clocks, tune)
                if c2.status() != 0:
                    raise SystemExit("a kernel reported a status: results are invalid")
                c2.close()
                r2.pop("out")
                entry = config_entry(wf, mf, r2, peak)
                torch.cuda.empty_cache()
            if frac == 0.0:
                zero_ms = entry["ms_per_step"]
            entry["measured_ratio"] = entry["ms_per_step"] / zero_ms
            fr.append(entry)
        configs["llama8b_by_fraction"] = fr
        wq = synth.WORKLOADS["qwen7b"]
        for name, wf in (("qwen7b_0pct", wq.with_(frac_compressed=0.0)), ("qwen7b", wq)):
            mf = synth.workload_mask(wf)
            c2, _, r2 = timed_steps(rl, harness, wf, mf, dev, stream, K, W, clocks, tune)
            if c2.status() != 0:
                raise SystemExit("a kernel reported a status: results are invalid")
            c2.close()
            r2.pop("out")
            configs[name] = config_entry(wf, mf, r2, peak)
            torch.cuda.empty_cache()
        configs["qwen7b"]["measured_ratio"] = configs["qwen7b"]["ms_per_step"] / configs["qwen7b_0pct"]["ms_per_step"]
        wc = synth.WORKLOADS["cot"]
        configs["cot_loop"] = run_loop(rl, harness, wc, synth.workload_mask(wc), dev, stream, clocks, args.loop_steps, peak)
        torch.cuda.empty_cache()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # ---- side measurement: mixed attention (Eq. 1) on a 4-layer all-full cache of the same shape.  Every
    # layer's K/V rows exceed the L2 and the launches cycle through the layers, so each launch reads from HBM.
    mixed = None
    if not args.no_mixed and world == 1:
        ml, reps = 4, max(K, 8)
        n = w.context + 1
        mw = w.with_(layers=ml, frac_compressed=0.0)
        mcache = harness.Cache(ml, w.kv_heads, w.q_heads, w.head_dim, w.batch, n + 8, np.ones(ml * w.kv_heads, np.uint8),
                               w.sink, w.window, device=dev)
        harness.fill_cache(mcache, mw, n)
        alpha = torch.rand(w.kv_heads, dtype=torch.float32, device=dev)
        q = q0
        mout = torch.empty((ml, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
        times = {}
        for name, call in (("plain", lambda l: rl.rlkv_decode_attention(mcache.handle, l, q[l % w.layers], mout[l], stream)),
                           ("mixed", lambda l: rl.rlkv_decode_mixed_attention(mcache.handle, l, q[l % w.layers], alpha,
                                                                              mout[l], stream))):
            for i in range(2 * ml):
                call(i % ml)
            torch.cuda.synchronize()
            e0.record(stream)
            for i in range(reps * ml):
                call(i % ml)
            e1.record(stream)
            torch.cuda.synchronize()
            times[name] = e0.elapsed_time(e1) / (reps * ml)
        full_bytes = w.batch * w.kv_heads * n * 4 * w.head_dim
        mixed = {"workload": f"{ml} all-full layers of the {w.name} shape, n = {n}, launches back to back (not overlapped)",
                 "launch_us": 1e3 * times["mixed"], "plain_launch_us": 1e3 * times["plain"],
                 "algorithmic_bytes_per_launch": full_bytes,
                 "achieved_gbs": full_bytes / (times["mixed"] * 1e-3) / 1e9,
                 "plain_gbs": full_bytes / (times["plain"] * 1e-3) / 1e9,
                 "rows_read_twice": 0, "launches_timed": reps * ml}
        if mcache.status() != 0:
            raise SystemExit("a mixed-attention kernel reported a status: results are invalid")
        mcache.close()
    # ---- side measurement: the paged, ragged cache on the first 4 layers of the workload's mask: the
    # same batch once with every sequence at the workload's length and once with lengths spread from
    # a quarter to seven quarters of it (same total), launches cycling through the layers
    paged = None
    if not args.no_paged and world == 1:
        pl, reps = w.layers, max(K, 8)
        n = w.context + 1
        pmask = mask[:pl * w.kv_heads]
        spread = harness.paged_spread_lengths(n, w.batch)
        paged = {"workload": f"the {pl} layers of the {w.name} mask, {w.batch} sequences; launch_us: rlkv_paged_decode_attention "
                             f"launches back to back; in_step: rlkv_paged_step (one append launch, one attention launch over all layers)"}
        variants = [("uniform", [n] * w.batch, False), ("ragged", spread, False)]
        if w.head_dim == 128:
            variants.append(("uniform_fp8", [n] * w.batch, True))   # every K/V row as an E4M3 code
        for name, lens, fp8 in variants:
            pages = sum((x + 63) // 64 for x in lens) + 2 + 2 * len(lens)
            scales = np.full(pl * w.kv_heads, 1.0 / 64, np.float32) if fp8 else None   # N(0,1) inputs stay well inside +-448
            pc = harness.PagedCache(pl, w.kv_heads, w.q_heads, w.head_dim, w.batch, pages, max(lens) + 128, pmask,
                                    w.sink, w.window, device=dev, k_scale=scales, v_scale=scales)
            slots = [pc.open_seq() for _ in lens]
            harness.fill_paged(pc, w, slots, lens)
            q = q0
            pout = torch.empty((pl, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
            lreps = max(2, (reps * 4) // pl)
            for i in range(pl):
                rl.rlkv_paged_decode_attention(pc.handle, i % pl, slots, q[i % pl], pout[i % pl], stream)
            torch.cuda.synchronize()
            e0.record(stream)
            for i in range(lreps * pl):
                rl.rlkv_paged_decode_attention(pc.handle, i % pl, slots, q[i % pl], pout[i % pl], stream)
            e1.record(stream)
            torch.cuda.synchronize()
            us = 1e3 * e0.elapsed_time(e1) / (lreps * pl)
            nbytes = sum(pc.step_bytes(l, slots) for l in range(pl)) / pl
            paged[name] = {"launch_us": us, "algorithmic_bytes_per_launch": nbytes, "achieved_gbs": nbytes / (us * 1e-6) / 1e9,
                           "lengths": [min(lens), max(lens)], "launches_timed": lreps * pl}
            # the same layers through rlkv_paged_step (one token appended per step, launches overlapped)
            kk, vv = kv0[0][:pl].contiguous(), kv0[1][:pl].contiguous()
            qq = q[:pl].contiguous()
            for i in range(3):
                rl.rlkv_paged_step(pc.handle, slots, kk, vv, qq, pout, stream)
            torch.cuda.synchronize()
            e0.record(stream)
            for i in range(reps):
                rl.rlkv_paged_step(pc.handle, slots, kk, vv, qq, pout, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            us = 1e3 * e0.elapsed_time(e1) / (reps * pl)
            nbytes = sum(pc.step_bytes(l, slots) for l in range(pl)) / pl
            paged[name]["in_step_us_per_layer"] = us
            paged[name]["in_step_gbs"] = nbytes / (us * 1e-6) / 1e9
            if pc.status() != 0:
                raise SystemExit("a paged decode kernel reported a status: results are invalid")
            pc.close()
    clocks.__exit__()

    # ---- CPU oracle on a bounded sample (rank 0, single-GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle.rlkv_oracle import max_threads
        oracle, step_in, sample_bytes, desc = build_oracle_sample(w, mask, dev)
        threads = max_threads()
        sec, reps = time_oracle(oracle, step_in, threads, 2, 3, min_seconds=10.0)
        sec1, reps1 = time_oracle(oracle, step_in, 1, 0, 1, min_seconds=5.0)
        total_bytes = workload_bytes(w, mask, w.context + 1)
        cpu = {"value": w.batch / (sec * total_bytes / sample_bytes), "unit": UNIT, "cores": threads,
               "kind": "oracle", "sample": f"{desc}; median of {reps} decodes, scaled to the step by K/V bytes",
               "single_thread_value": w.batch / (sec1 * total_bytes / sample_bytes),
               "oracle_gbs": sample_bytes / sec / 1e9, "host": host_description()}

    if rank == 0:
        total_bytes = res["kv_bytes_per_step"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": median_ms, "ms_per_step_mean": mean_ms,
            "ms_per_step_min_max": [res["ms_per_step_min"], res["ms_per_step_max"]],
            "value_from": "median of the K per-step times (one CUDA event between consecutive steps)",
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": config_dict(w, mask),
            "kv_bytes_per_step": total_bytes,
            "step_hbm_gbs": total_bytes / (median_ms * 1e-3) / 1e9,
            "bytes_ratio_vs_uncompressed": total_bytes / (w.batch * w.layers * w.kv_heads * (w.context + W + 1 + K // 2) * 4 * w.head_dim),
            "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "gpu_launches": launches,
            "per_layer_calls": per_layer, "configs": configs, "mixed_attention": mixed, "paged_cache": paged,
            "clocks": main_clocks,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main(argv=None):
    args = parse_args(argv)
    if args.sweep_table:
        sweep_table(args.sweep_table)
        return
    w = pick_workload(args)
    mask = synth.workload_mask(w)
    if args.impl == "reference":
        run_reference(args, w, mask)
    else:
        run_ours(args, w, mask)


if __name__ == "__main__":
    main()
