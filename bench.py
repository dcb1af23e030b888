#!/usr/bin/env python
"""Benchmark of the per-chunk KV-cache codec on the five seeded synthetic workloads.

  python bench.py [--workload W] [--gpus N] [--steps K] [--warmup W]     the CUDA library
  python bench.py --impl reference ...                                   the CPU oracle, as it stands

Workloads (--workload; the default is the 70B-shaped context, the one the target is quoted on):
  tiny             l=4,  N=256     one chunk; 4 MiB of KV, so L2 is flushed between launches and the
                                   figures are launch latencies, not HBM rates
  llama3-8b-8k     l=32, N=8192    every chunk at each level in turn
  batch-64         64 contexts of the 8B shape, lengths log-uniform in [2K, 32K], a random level per
                                   chunk, one shared pool behind one shuffled page table: the step is
                                   ONE batched decode launch over all chunks (the contexts are encoded
                                   once during set-up: their bf16 sources do not fit beside the pool)
  llama3-70b-32k   l=80, N=32768   one level per launch over all levels
  llama3-8b-128k   l=32, N=131072  encode of the full context then decode-to-pages at every level,
                                   the two directions timed as adjacent event intervals

One step = one pass of the whole hot path over the workload: for every level in turn, size
arithmetic (host), encode of the context into its stored form, batched decode of all chunks into a
paged bf16 pool through a shuffled page table.  Inputs are resident in HBM when the timed region
starts.

Prints one JSON line (rank 0).  `value` is decode throughput in GB/s of bf16 written (bytes decoded
over the sum of the decode intervals inside the timed steps); `roofline` relates the decode kernel's
algorithmic HBM bytes to the measured copy bandwidth; `e2e` is the same metric with the stored form
in pinned host memory (PCIe copy and status read-back inside the timed interval); `cpu_baseline`
times the oracle on the host cores; `level_stats` repeats every launch of a step many times on its
own, with the SM clock sampled meanwhile, and gives time x clock per launch so that a change of the
kernel can be told from a change of the clock.

With --gpus N > 1 and no launcher around it, the script starts its own N ranks (one per GPU,
independent replicas: the codec has no exchange step).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Callable, Optional

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import workloads

METRIC = "KV decode GB/s (bf16 out)"
UNIT = "GB/s"
LEVELS = (0, 1, 2, 3)
CODE_BITS = {0: 16, 1: 8, 2: 4, 3: 2}
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 << 20

SHAPES = {s.name: s for s in (workloads.TINY, workloads.LLAMA8B_8K, workloads.LLAMA70B_32K, workloads.LLAMA8B_128K)}
BATCH = "batch-64"
WORKLOAD_NAMES = ["tiny", "llama3-8b-8k", BATCH, "llama3-70b-32k", "llama3-8b-128k"]

# DRAM bytes of one launch relative to its algorithmic bytes (dram__bytes_read.sum +
# dram__bytes_write.sum of an ncu capture on a 4096-token slice of the 70B-shaped workload; traffic
# grows in proportion to the tokens, every element being touched once).  The ratios hold for the
# kernel sources with the digest recorded beside them (kernel_source_digest()); once a kernel source
# has changed, `traffic` is reported as null until the capture is repeated.
TRAFFIC = {
    "captured": "2026-11-28",
    "source_digest": "ca5950608c05f5a8",
    "decode": {0: 0.9801, 1: 0.9724, 2: 0.9673, 3: 0.9630},
    "encode": {0: 0.9792, 1: 0.9795, 2: 0.9865, 3: 0.9919},
    # executed thread instructions per element of the transcoding instances whose source is quantised
    # (smsp__inst_executed.sum x 32 / elements of the same capture): these are bound by instruction
    # issue, not by memory
    "transcode_instr": {(1, 2): 8.22, (1, 3): 8.24, (2, 3): 8.42},
}
ISSUE_LANES_PER_SM = 4 * 32      # four schedulers per SM, one warp instruction (32 threads) per clock each


def kernel_source_digest() -> str:
    """SHA-256 over the kernel sources of the library (what the DRAM-traffic ratios depend on)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2509_00105_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")):
            with open(os.path.join(csrc, name), "rb") as f:
                h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()[:16]


def measured_peak() -> tuple[float, str]:
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(elements: int, stream_bytes: int) -> int:
    """Bytes one launch must move: the stored stream on one side, 2 bytes per element on the other."""
    return stream_bytes + 2 * elements


def pci_bus_id(device_index: int) -> Optional[str]:
    """PCI bus id of a CUDA device, the one name nvidia-smi and NVML share with the CUDA runtime
    whatever CUDA_VISIBLE_DEVICES says."""
    try:
        p = torch.cuda.get_device_properties(device_index)
        return f"{p.pci_domain_id:08x}:{p.pci_bus_id:02x}:{p.pci_device_id:02x}.0"
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu: str):
        self.gpu = gpu
        self.proc = None
        self.lines: list[str] = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", self.gpu], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line)

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        note = None
        if not self.lines:                               # the region was shorter than one sampling period: one reading now
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-i", self.gpu],
                                     capture_output=True, text=True, timeout=10).stdout
                self.lines = out.splitlines()
                note = "timed region shorter than the sampling period: one reading taken right after it"
            except (OSError, subprocess.TimeoutExpired):
                pass
        sm, mx, power, reasons = [], [], [], set()
        for line in self.lines:
            p = [x.strip() for x in line.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2])); power.append(float(p[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        out = {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
               "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}
        if note:
            out["note"] = note
        return out


class NvmlClock:
    """Reads the SM clock of one GPU through NVML every few milliseconds from a thread (reading
    only; nothing is ever set).  Used for the short per-launch statistics, where nvidia-smi's
    sampling period is too coarse."""

    def __init__(self, bus_id: Optional[str]):
        self.handle = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByPciBusId(bus_id.encode()) if bus_id else None
        except Exception:
            self.handle = None
        self.samples: list[float] = []
        self._stop = threading.Event()
        self._thread = None

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(float(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM)))
            except Exception:
                return
            time.sleep(0.004)

    def start(self):
        self.samples = []
        self._stop.clear()
        if self.handle is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self) -> Optional[float]:
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
            self._thread = None
        return statistics.median(self.samples) if self.samples else None


# ------------------------------------------------------------------------------------------
# the CPU oracle as a timed baseline (also the `--impl reference` arm)
# ------------------------------------------------------------------------------------------

def oracle_sample_step(kv_np: np.ndarray, n_threads: int) -> tuple[float, float, int]:
    """Encode then decode one 256-token chunk per thread at every level with the oracle.
    kv_np: uint16 [l_s][2][256 * n_threads][c].  Returns (encode_s, decode_s, elements_per_level)."""
    import oracle
    l, _, N, c = kv_np.shape
    enc_s = dec_s = 0.0
    elements = l * 2 * N * c
    ids = np.arange(16, dtype=np.int32)
    pools = [np.empty(l * 2 * 16 * 16 * c, dtype=np.uint16) for _ in range(n_threads)]
    with ThreadPoolExecutor(n_threads) as ex:
        for level in LEVELS:
            t = time.perf_counter()
            streams = list(ex.map(lambda i: oracle.encode_chunk(kv_np, 256 * i, 256, level), range(n_threads)))
            enc_s += time.perf_counter() - t
            t = time.perf_counter()
            list(ex.map(lambda i: oracle.decode_chunk(streams[i], level, l, c, 256, ids, pools[i], 2 * 16 * 16 * c,
                                                      16 * 16 * c, 16 * c, 16), range(n_threads)))
            dec_s += time.perf_counter() - t
    return enc_s, dec_s, elements


def oracle_inputs(n_layers: int, n_channels: int, n_threads: int, target_s: float):
    """A slice of the workload (some layers, one chunk per thread) sized to about target_s per step."""
    import oracle
    oracle.build()
    probe = workloads.make_kv(1, 256 * n_threads, n_channels, seed=4000)
    probe_np = probe.view(torch.int16).numpy().view(np.uint16)
    e, d, _ = oracle_sample_step(probe_np, n_threads)
    layers = max(1, min(n_layers, int(target_s / max(e + d, 1e-3))))
    kv = workloads.make_kv(layers, 256 * n_threads, n_channels, seed=4000)
    return kv.view(torch.int16).numpy().view(np.uint16), layers


def workload_config(name: str, tokens: int = 0) -> dict:
    """The `config` object of the JSON line: what the workload is, without any device work."""
    if name == BATCH:
        lengths = workloads.context_lengths(workloads.BATCH_N_CONTEXTS, workloads.BATCH_MIN_TOKENS,
                                            workloads.BATCH_MAX_TOKENS, seed=3000)
        return {"workload": name, "n_layers": workloads.LLAMA8B_8K.n_layers, "n_channels": 1024,
                "n_contexts": len(lengths), "n_tokens": sum(lengths), "chunk_tokens": 256, "page_tokens": 16,
                "levels": "uniformly random per chunk",
                "step": "one batched decode-to-pages launch over every chunk of the 64 contexts"}
    s = SHAPES[name]
    n = tokens or s.n_tokens
    return {"workload": name if not tokens else f"{name}-first{tokens}", "n_layers": s.n_layers,
            "n_channels": s.n_channels, "n_tokens": n, "chunk_tokens": 256, "page_tokens": 16, "levels": list(LEVELS),
            "step": "encode + batched decode-to-pages at every level"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return                                           # one CPU program: rank 0 alone runs it
    cfg = workload_config(args.workload, args.tokens)
    cores = len(os.sched_getaffinity(0))
    kv_np, layers = oracle_inputs(cfg["n_layers"], cfg["n_channels"], cores, target_s=1.5)
    for _ in range(args.warmup):
        oracle_sample_step(kv_np, cores)
    enc = dec = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e, d, elements = oracle_sample_step(kv_np, cores)
        enc += e; dec += d
    total = time.perf_counter() - t0
    value = len(LEVELS) * 2 * elements * args.steps / dec / 1e9
    sample = f"{layers} of {cfg['n_layers']} layers x {cores} chunks of 256 tokens, every level, per step"
    cfg["sample"] = sample
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": cfg,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                         "encode_gbps_bf16_in": len(LEVELS) * 2 * elements * args.steps / enc / 1e9},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------
# the CUDA library
# ------------------------------------------------------------------------------------------

def rank_seed(rank: int) -> int:
    """Every rank encodes and loads a context of its own (weak scaling: replicas, no exchange)."""
    return 3000 + rank


def max_over_ranks(values: list[float], device, world: int) -> list[float]:
    """Element-wise maximum of per-rank timings: the job is as slow as its slowest rank."""
    if world == 1:
        return list(values)
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_gbps(world: int, bytes_per_rank: float, ms: float) -> float:
    """Aggregate throughput of `world` ranks that each moved bytes_per_rank in (at most) ms."""
    return world * bytes_per_rank / ms / 1e6


@dataclass
class Leg:
    """One (encode, decode) pair of a step: a level of a context, or the mixed batch."""
    name: str
    level: Optional[int]              # None: a mix of levels
    elements: int                     # bf16 elements decoded
    tokens: int
    stream_bytes: int
    encode: Optional[Callable[[], None]]
    decode: Callable[[], None]


class ContextWorkload:
    """One context of a fixed shape: every level in turn, encode then decode."""

    def __init__(self, kvh, name, shape, dev, seed):
        self.kvh, self.name, self.dev = kvh, name, dev
        l, c, N = shape.n_layers, shape.n_channels, shape.n_tokens
        self.l, self.c, self.N = l, c, N
        self.n_chunks = workloads.n_chunks(N)
        n_pages = workloads.n_pages(N)
        self.kv = workloads.make_kv(l, N, c, seed=seed, device=dev)       # every rank its own context
        self.pool = kvh.Pool.allocate(l, n_pages, c, device=dev)
        self.table = workloads.shuffled_page_table(n_pages, n_pages, seed=seed).to(dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.plans = {}
        for level in LEVELS:
            descs, total = kvh.plan_chunks(l, c, N, level)
            assert total == sum(kvh.level_bytes(level, l, c, int(n)) for n in descs["n_tok"])
            self.plans[level] = (descs, kvh.descs_to_tensor(descs, dev), total)
        self.stream_buf = torch.empty(max(p[2] for p in self.plans.values()), dtype=torch.uint8, device=dev)
        self.footprint = 2 * self.kv.numel() * 2 + self.stream_buf.numel()
        self.legs = [self._leg(level) for level in LEVELS]

    def _leg(self, level):
        kvh = self.kvh
        descs, descs_dev, total = self.plans[level]
        return Leg(f"L{level}", level, self.l * 2 * self.N * self.c, self.N, total,
                   lambda: kvh.encode(self.kv, level, out=self.stream_buf[:total], dev_status=self.status),
                   lambda: kvh.decode_batch(self.stream_buf[:total], descs_dev, self.n_chunks, self.table, self.pool,
                                            self.status))

    # ---- end to end: the stored form lives in pinned host memory -----------------------------
    def e2e_setup(self):
        self.host = torch.empty(self.stream_buf.numel(), dtype=torch.uint8).pin_memory()

    def e2e_leg(self, leg, host_status, copy_stream):
        """(store, load) callables of one leg."""
        descs, descs_dev, _ = self.plans[leg.level]
        kvh = self.kvh
        return (lambda: kvh.store_host(self.kv, descs, descs_dev, self.stream_buf, self.host, self.status, host_status,
                                       copy_stream),
                lambda: kvh.load_host(self.host, self.stream_buf, descs, descs_dev, self.table, self.pool, self.status,
                                      host_status, copy_stream))


class BatchWorkload:
    """64 contexts of the 8B shape with a level per chunk, decoded into one shared pool in one launch."""

    def __init__(self, kvh, name, dev, seed, n_layers=None):
        self.kvh, self.name, self.dev = kvh, name, dev
        c = 1024
        lengths = workloads.context_lengths(workloads.BATCH_N_CONTEXTS, workloads.BATCH_MIN_TOKENS,
                                            workloads.BATCH_MAX_TOKENS, seed=seed)
        levels = [workloads.chunk_levels(workloads.n_chunks(N), 4, seed=seed + 100 + i) for i, N in enumerate(lengths)]
        l = n_layers or workloads.LLAMA8B_8K.n_layers
        self.l, self.c, self.N = l, c, sum(lengths)
        total_pages = sum(workloads.n_pages(n) for n in lengths)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        plans, total_bytes, pt_base = [], 0, 0
        for N, lv in zip(lengths, levels):
            descs, size = kvh.plan_chunks(l, c, N, lv, stream_base=total_bytes, pt_base=pt_base)
            plans.append(descs)
            total_bytes += size
            pt_base += workloads.n_pages(N)
        self.descs = np.concatenate(plans)
        self.descs_dev = kvh.descs_to_tensor(self.descs, dev)
        self.blob = torch.empty(total_bytes, dtype=torch.uint8, device=dev)
        for i, (N, descs) in enumerate(zip(lengths, plans)):              # set-up: the stored form of every context
            kv = workloads.make_kv(l, N, c, seed=seed + 200 + i, device=dev)
            local = descs.copy()
            base = int(descs["stream_off"][0])
            local["stream_off"] -= base
            size = int(local["stream_off"][-1]) + kvh.level_bytes(int(local["level"][-1]), l, c, int(local["n_tok"][-1]))
            kvh.encode_chunks(kv, kvh.descs_to_tensor(local, dev), len(local), self.blob[base:base + size], self.status,
                              descs=local)
            del kv
        self.pool = kvh.Pool.allocate(l, total_pages, c, device=dev)
        self.table = workloads.shuffled_page_table(total_pages, total_pages, seed=seed + 1).to(dev)
        self.n_chunks = len(self.descs)
        self.footprint = self.blob.numel() + self.pool.tensor.numel() * 2
        self.legs = [Leg("mixed", None, l * 2 * self.N * c, self.N, total_bytes, None,
                         lambda: kvh.decode_batch(self.blob, self.descs_dev, self.n_chunks, self.table, self.pool,
                                                  self.status))]
        self.level_share = {k: float(np.mean(self.descs["level"] == k)) for k in LEVELS}

    def e2e_setup(self):
        self.host = torch.empty(self.blob.numel(), dtype=torch.uint8).pin_memory()
        step = 1 << 30
        for off in range(0, self.blob.numel(), step):
            self.host[off:off + step].copy_(self.blob[off:off + step])
        torch.cuda.synchronize()

    def e2e_leg(self, leg, host_status, copy_stream):
        kvh = self.kvh
        return (None, lambda: kvh.load_host(self.host, self.blob, self.descs, self.descs_dev, self.table, self.pool,
                                            self.status, host_status, copy_stream))


def timed_launches(fn, reps: int, flush=None):
    """Per-launch times (ms) of `reps` launches of fn, each between its own pair of events."""
    pairs = []
    for _ in range(reps):
        if flush is not None:
            flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        pairs.append((a, b))
    torch.cuda.synchronize()
    return sorted(a.elapsed_time(b) for a, b in pairs)


def level_statistics(w, clock: NvmlClock, reps: int, flush, peak: float) -> list[dict]:
    """Every launch of a step on its own, `reps` times back to back, with the SM clock sampled
    meanwhile: median and minimum time, the clock's median, and their product (time x clock, in
    ms x MHz = thousands of SM cycles), which stays put when only the clock moves."""
    out = []
    for leg in w.legs:
        for kind, fn in (("encode", leg.encode), ("decode", leg.decode)):
            if fn is None:
                continue
            fn()
            torch.cuda.synchronize()
            clock.start()
            t = timed_launches(fn, reps, flush)
            mhz = clock.stop()
            med = statistics.median(t)
            alg = algorithmic_bytes(leg.elements, leg.stream_bytes)
            out.append({"leg": leg.name, "kind": kind, "launches": reps, "ms_median": round(med, 4), "ms_min": round(t[0], 4),
                        "sm_mhz_median": mhz, "ms_x_mhz": round(med * mhz, 1) if mhz else None,
                        "hbm_gbps_median": round(alg / med / 1e6, 1), "roofline_frac_median": round(alg / med / 1e6 / peak, 4)})
    return out


def time_extras(kvh, w, clock: "NvmlClock", sms: int, instr_ok: bool, reps: int = 20):
    """Transcoding (every pair of levels) and token dropping (4 sink tokens + a recent window, a
    quarter of the context kept), each as the mean of `reps` launches over the whole context after
    one warm-up launch.  Bytes counted: streams read + streams written (transcode), kept bf16 rows
    read + streams written (token dropping).  Transcoding from a quantised source is bound by
    instruction issue: its line carries an "alu" roofline too, the time the counted thread
    instructions per element need at one warp instruction per scheduler and clock, at the SM clock
    sampled during the launches."""
    def timed(fn):
        fn()
        clock.start()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        b.synchronize()
        return a.elapsed_time(b) / reps, clock.stop()

    l, c, N = w.l, w.c, w.N
    elements = l * 2 * N * c
    out = {"transcode": [], "token_dropping": []}
    second = torch.empty(w.plans[1][2], dtype=torch.uint8, device=w.dev)
    for lin in (0, 1, 2):
        _, descs_in_dev, total_in = w.plans[lin]
        kvh.encode(w.kv, lin, out=w.stream_buf[:total_in], dev_status=w.status)
        for lout in range(lin + 1, 4):
            _, descs_out_dev, total_out = w.plans[lout]
            ms, mhz = timed(lambda: kvh.transcode(w.stream_buf[:total_in], descs_in_dev, second[:total_out], descs_out_dev,
                                                  w.n_chunks, l, c, lin, lout, dev_status=w.status))
            row = {"from": lin, "to": lout, "ms": round(ms, 4), "hbm_gbps": round((total_in + total_out) / ms / 1e6, 1),
                   "tokens_per_s": round(N / ms * 1e3)}
            per_el = TRAFFIC["transcode_instr"].get((lin, lout))
            if per_el and instr_ok and mhz:
                bound_ms = elements * per_el / (sms * ISSUE_LANES_PER_SM * mhz * 1e3)
                row["roofline_alu"] = {"bound": "alu", "thread_instr_per_element": per_el, "sm_mhz": mhz,
                                       "peak": round(sms * ISSUE_LANES_PER_SM * mhz / 1e6, 2), "unit": "T thread-instr/s",
                                       "achieved": round(elements * per_el / ms / 1e9, 2), "bound_ms": round(bound_ms, 4),
                                       "frac": round(bound_ms / ms, 4)}
            out["transcode"].append(row)
    # a level per chunk (uniformly random): the general encoder instance over device descriptors alone, and the
    # per-level instances when the caller also passes its host copy of the descriptors
    lv = workloads.chunk_levels(w.n_chunks, 4, seed=77)
    mdescs, mtotal = kvh.plan_chunks(l, c, N, lv)
    mdev = kvh.descs_to_tensor(mdescs, w.dev)
    out["encode_mixed_levels"] = {}
    for key, host in (("device_descriptors_only", None), ("with_host_descriptors", mdescs)):
        ms, _ = timed(lambda: kvh.encode_chunks(w.kv, mdev, len(mdescs), w.stream_buf[:mtotal], w.status, descs=host))
        out["encode_mixed_levels"][key] = {"ms": round(ms, 4), "hbm_gbps": round((2 * elements + mtotal) / ms / 1e6, 1)}
    runs, n_kept = kvh.keep_sinks_and_recent(N, 4, max(N // 4 - 4, 1))
    for level in LEVELS:
        descs, total = kvh.plan_chunks(l, c, n_kept, level)
        ms, _ = timed(lambda: kvh.encode_kept(w.kv, runs, None, len(descs), second[:total], w.status, level=level))
        out["token_dropping"].append({"level": level, "kept_tokens": n_kept, "ms": round(ms, 4),
                                      "hbm_gbps": round((2 * elements * n_kept // N + total) / ms / 1e6, 1)})
    assert w.status.item() == 0
    return out


def mix_ceiling(w, reps: int = 10):
    """What kernels that do no codec work reach at the read : write mix of each level's decode
    launch, on the same amount of data: a plain grid-stride loop of 16-byte loads and stores, a
    loop of bulk copies through shared memory (no per-element instructions at all; with a fixed
    stride and with units handed out dynamically), and the decode
    kernel's own skeleton (producer warp, two-stage ring, 8 consumer warps, dynamic hand-out of
    units, the same store pattern) with the codec taken out, writing its pages in order and to
    pseudo-random pages of the destination as a shuffled page table makes the decoder do.  Not bounds, but they show how much of
    a level's distance from the copy peak belongs to the memory system's handling of write-heavy
    streams, and the last one what the arithmetic costs on top of moving the bytes."""
    import ctypes
    from paper_2509_00105_b200 import _build
    L = ctypes.CDLL(str(_build.build(variant="probe")))
    L.kvh_probe_stream_mix.restype = ctypes.c_int
    L.kvh_probe_stream_mix.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int,
                                       ctypes.c_void_p, ctypes.c_void_p]
    dst = w.pool.tensor
    out = []
    for leg in w.legs:
        if leg.level is None:
            continue
        reads16 = {0: 16, 1: 9, 2: 5, 3: 3}[leg.level]           # 16-byte reads per 16 16-byte writes
        write_bytes = (2 * leg.elements) // 65536 * 65536
        row = {"level": leg.level, "read_write": f"{reads16}:16"}
        for kind, name in ((0, "ldst"), (1, "bulk"), (3, "bulk_dyn"), (2, "ring"), (4, "ring_scatter")):
            def fn():
                st = L.kvh_probe_stream_mix(kind, w.kv.data_ptr(), dst.data_ptr(), write_bytes, reads16,
                                            w.status.data_ptr(), torch.cuda.current_stream().cuda_stream)
                assert st == 0, st
            fn()
            t = timed_launches(fn, reps)
            row[f"{name}_ms_median"] = round(statistics.median(t), 4)
            row[f"{name}_hbm_gbps"] = round(write_bytes * (16 + reads16) / 16 / statistics.median(t) / 1e6, 1)
        out.append(row)
    assert w.status.item() == 0
    return out


def run_ours(args):
    import torch.distributed as dist
    import paper_2509_00105_b200 as pkg

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert world == args.gpus, f"--gpus {args.gpus} but the launcher started {world} ranks"
    assert torch.cuda.is_available() and torch.cuda.device_count() > local, "no CUDA device for this rank"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    kvh = pkg.variant(args.variant)                      # fails loudly if the extension is missing
    kvh.lib()

    cfg = workload_config(args.workload, args.tokens)
    if args.workload == BATCH:
        w = BatchWorkload(kvh, args.workload, dev, seed=rank_seed(rank))
    else:
        shape = SHAPES[args.workload]
        if args.tokens:
            shape = workloads.Shape(cfg["workload"], shape.n_layers, shape.n_channels, args.tokens)
        w = ContextWorkload(kvh, cfg["workload"], shape, dev, seed=rank_seed(rank))
    status = w.status
    small = w.footprint < 2 * L2_BYTES                   # would sit in L2 from one launch to the next
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if small else None
    flush = (lambda: flush_buf.fill_(1)) if small else None

    def step(events=None):
        for i, leg in enumerate(w.legs):
            ev = events[i] if events is not None else None
            if leg.encode is not None:
                if flush: flush()
                if ev: ev[0].record()
                leg.encode()
                if ev: ev[1].record()
            if flush: flush()
            if ev: ev[2].record()
            leg.decode()
            if ev: ev[3].record()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 0)):
        step()
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in w.legs] for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    bus = pci_bus_id(local)
    sampler = ClockSampler(bus or str(local))
    barrier()
    sampler.start()
    t_start.record()
    for s in range(args.steps):
        step(ev[s])
    t_end.record()
    barrier()
    clocks = sampler.stop()
    assert status.item() == 0, f"device status {status.item()}"

    n_legs = len(w.legs)
    total_ms = t_start.elapsed_time(t_end)
    enc_all = [sorted(e[i][0].elapsed_time(e[i][1]) for e in ev) if w.legs[i].encode else [] for i in range(n_legs)]
    dec_all = [sorted(e[i][2].elapsed_time(e[i][3]) for e in ev) for i in range(n_legs)]
    enc_ms = [sum(x) / args.steps if x else 0.0 for x in enc_all]
    dec_ms = [sum(x) / args.steps for x in dec_all]
    times = max_over_ranks([total_ms] + enc_ms + dec_ms, dev, world)
    total_ms, enc_ms, dec_ms = times[0], times[1:1 + n_legs], times[1 + n_legs:]

    peak, peak_kind = measured_peak()
    single = world == 1

    # ---- each launch of a step on its own, with the clock: time x clock per level ----
    level_stats = None
    if single and args.stat_launches > 0:
        level_stats = level_statistics(w, NvmlClock(bus), args.stat_launches, flush, peak)

    # ---- the two further store-side operations and the plain-streaming ceilings ----
    extras = None
    if single and not args.no_extras and isinstance(w, ContextWorkload):
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        extras = time_extras(kvh, w, NvmlClock(bus), sms, TRAFFIC["source_digest"] == kernel_source_digest() and w.c == 1024,
                             reps=args.extras_reps)
        extras["mix_ceiling"] = mix_ceiling(w)

    # ---- end to end: stored form in pinned host memory ----
    e2e = None
    if not args.no_e2e:
        w.e2e_setup()
        host_status = torch.zeros(1, dtype=torch.int32).pin_memory()
        copy_stream = torch.cuda.Stream(device=dev)
        main_stream = torch.cuda.Stream(device=dev)
        k_e2e = max(1, min(args.steps, args.e2e_steps))
        load_ms = [0.0] * n_legs
        store_ms = [0.0] * n_legs
        with torch.cuda.stream(main_stream):
            for it in range(1 + k_e2e):                  # one untimed pass first
                for i, leg in enumerate(w.legs):
                    store, load = w.e2e_leg(leg, host_status, copy_stream)
                    a, b, d = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                    a.record()
                    if store is not None:
                        store()
                    b.record()
                    load()
                    d.record()
                    d.synchronize()
                    assert host_status.item() == 0
                    if it > 0:
                        store_ms[i] += a.elapsed_time(b) / k_e2e
                        load_ms[i] += b.elapsed_time(d) / k_e2e
        t = max_over_ranks(load_ms + store_ms, dev, world)
        load_ms, store_ms = t[:n_legs], t[n_legs:]
        stream_total = sum(leg.stream_bytes for leg in w.legs)
        has_store = any(leg.encode is not None for leg in w.legs)
        bf16_bytes = sum(2 * leg.elements for leg in w.legs)
        e2e = {"value": whole_job_gbps(world, bf16_bytes, sum(load_ms)), "unit": UNIT,
               "h2d_bytes_per_step": stream_total,
               "d2h_bytes_per_step": (stream_total if has_store else 0) + 4 * (2 if has_store else 1) * n_legs,
               "steps": k_e2e, "what": "kvh_load_host: pinned host streams -> HBM -> pages, status read back",
               "load_ms_per_leg": [round(x, 3) for x in load_ms]}
        if has_store:
            e2e["store_ms_per_leg"] = [round(x, 3) for x in store_ms]
            e2e["store_gbps_bf16_in"] = whole_job_gbps(world, bf16_bytes, sum(store_ms))
        del w.host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    mhz = clocks.get("sm_mhz")
    legs_out = []
    for i, leg in enumerate(w.legs):
        alg = algorithmic_bytes(leg.elements, leg.stream_bytes)
        row = {"leg": leg.name, "level": leg.level, "bits": CODE_BITS.get(leg.level), "stream_bytes": leg.stream_bytes,
               "decode_ms": round(dec_ms[i], 4), "decode_ms_median": round(statistics.median(dec_all[i]), 4),
               "decode_ms_min": round(dec_all[i][0], 4),
               "decode_gbps_bf16_out": round(2 * leg.elements / dec_ms[i] / 1e6, 1),
               "decode_hbm_gbps": round(alg / dec_ms[i] / 1e6, 1),
               "decode_roofline_frac": round(alg / dec_ms[i] / 1e6 / peak, 4),
               "decode_tokens_per_s": round(leg.tokens / dec_ms[i] * 1e3),
               "decode_ms_x_mhz": round(statistics.median(dec_all[i]) * mhz, 1) if mhz else None}
        if leg.encode is not None:
            row.update({"encode_ms": round(enc_ms[i], 4), "encode_ms_median": round(statistics.median(enc_all[i]), 4),
                        "encode_ms_min": round(enc_all[i][0], 4), "encode_hbm_gbps": round(alg / enc_ms[i] / 1e6, 1),
                        "encode_roofline_frac": round(alg / enc_ms[i] / 1e6 / peak, 4),
                        "encode_ms_x_mhz": round(statistics.median(enc_all[i]) * mhz, 1) if mhz else None})
        legs_out.append(row)
    dec_total_ms = sum(dec_ms)
    enc_total_ms = sum(enc_ms)
    alg_total = sum(algorithmic_bytes(leg.elements, leg.stream_bytes) for leg in w.legs)
    bf16_total = sum(2 * leg.elements for leg in w.legs)
    achieved = alg_total / dec_total_ms / 1e6

    # DRAM traffic per launch: the captured ratios, if they still describe these kernels
    digest = kernel_source_digest()
    traffic_ok = TRAFFIC["source_digest"] == digest and w.c == 1024 and not small

    def traffic(kind):
        if not traffic_ok:
            return None
        if isinstance(w, BatchWorkload):                 # a mix: every level by its share of the chunks' bytes
            by_level = {k: 0 for k in LEVELS}
            for d in w.descs:
                n_el = w.l * 2 * int(d["n_tok"]) * w.c
                by_level[int(d["level"])] += algorithmic_bytes(n_el, kvh.level_bytes(int(d["level"]), w.l, w.c, int(d["n_tok"])))
            return sum(TRAFFIC[kind][k] * b for k, b in by_level.items())
        return sum(TRAFFIC[kind][leg.level] * algorithmic_bytes(leg.elements, leg.stream_bytes) for leg in w.legs) / n_legs

    cfg.update({"l2": ("L2 flushed (a 252 MiB fill) before every launch: the workload is smaller than L2" if small else
                       f"inputs larger than L2 ({w.footprint / 1e9:.1f} GB touched per step)"),
                "parallelism": f"replicas x{world}", "library_build": kvh.build_variant()})
    if isinstance(w, BatchWorkload):
        cfg["n_chunks"] = w.n_chunks
        cfg["level_share_of_chunks"] = {str(k): round(v, 3) for k, v in w.level_share.items()}
    launches_per_step = sum(2 if leg.encode is not None else 1 for leg in w.legs)
    out = {
        "metric": METRIC, "value": whole_job_gbps(world, bf16_total, dec_total_ms), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": cfg,
        "decode_ms_per_step": dec_total_ms, "encode_ms_per_step": enc_total_ms,
        "tokens_per_s_loaded": world * sum(leg.tokens for leg in w.legs) / dec_total_ms * 1e3,
        "levels": legs_out,
        "roofline": {"bound": "hbm", "kernel": "decode_tma_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic("decode"), "peak_kind": f"of {peak_kind}",
                     "traffic_kind": (f"ncu capture of {TRAFFIC['captured']} on a 4096-token slice, scaled by tokens"
                                      if traffic_ok else "none for these kernel sources"),
                     "frac_of_8TBs_datasheet": achieved / 8000.0,
                     "per_launch": f"mean over the {n_legs} decode launch(es) of a step: stream bytes + 2 B/element"},
        "gpu_launches": args.steps * launches_per_step,
        "kernel_source_digest": digest,
        "clocks": clocks,
    }
    if enc_total_ms > 0:
        out["roofline_encode"] = {"bound": "hbm", "kernel": "encode_tma_kernel", "achieved": alg_total / enc_total_ms / 1e6,
                                  "peak": peak, "unit": "GB/s", "frac": alg_total / enc_total_ms / 1e6 / peak,
                                  "traffic": traffic("encode"), "peak_kind": f"of {peak_kind}",
                                  "per_launch": f"mean over the {n_legs} encode launches of a step: 2 B/element + stream bytes"}
    if level_stats is not None:
        out["level_stats"] = level_stats
    if e2e is not None:
        out["e2e"] = e2e
    if extras is not None:
        for key in ("transcode", "token_dropping"):
            for r in extras[key]:
                r["roofline_frac"] = round(r["hbm_gbps"] / peak, 4)
        for r in extras["encode_mixed_levels"].values():
            r["roofline_frac"] = round(r["hbm_gbps"] / peak, 4)
        out["extras"] = extras
    if single and not args.no_cpu_baseline:
        cores = len(os.sched_getaffinity(0))
        kv_np, layers = oracle_inputs(w.l, w.c, cores, target_s=4.0)
        e, d, el = oracle_sample_step(kv_np, cores)
        one_np = np.ascontiguousarray(kv_np[:max(1, kv_np.shape[0] // 8), :, :256])     # one chunk, an eighth of the layers
        e1, d1, el1 = oracle_sample_step(one_np, 1)
        out["cpu_baseline"] = {
            "single_thread_value": len(LEVELS) * 2 * el1 / d1 / 1e9,
            "value": len(LEVELS) * 2 * el / d / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{layers} of {w.l} layers x {cores} chunks of 256 tokens, every level, encode {e:.1f} s + decode {d:.1f} s",
            "encode_gbps_bf16_in": len(LEVELS) * 2 * el / e / 1e9}
        # the sample's rates applied to the whole step: not measured
        full = sum((2.0 if leg.encode is not None else 1.0) * leg.elements for leg in w.legs)
        out["cpu_baseline"]["extrapolated_step_s"] = round(full / (len(LEVELS) * 2 * el) * (e + d), 1)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_policy(args):
    """Time the greedy policy (host C++) on synthetic entries: 16 stored forms per entry (4 levels x 4
    kept fractions of the tokens), sizes from the library's own size arithmetic for the 8B shape,
    capacity an eighth of the full-quality total.  One host core; no GPU work."""
    import paper_2509_00105_b200 as kvh
    n = args.policy_entries
    l, c = workloads.LLAMA8B_8K.n_layers, 1024
    rng = np.random.default_rng(7)
    freq = 10.0 / (rng.permutation(n) + 1.0)
    tokens = np.exp(rng.uniform(np.log(workloads.BATCH_MIN_TOKENS), np.log(workloads.BATCH_MAX_TOKENS), n)).astype(np.int64)
    forms = [(level, keep) for keep in (1.0, 0.5, 0.25, 0.125) for level in range(4)]
    chunk = {k: np.array([0] + [kvh.level_bytes(k, l, c, t) for t in range(1, 257)], dtype=np.int64) for k in range(4)}
    sens_q, sens_d = 0.02 + 0.25 * rng.random(n), 0.05 + 0.9 * rng.random(n)
    options = np.empty(n * len(forms), dtype=kvh.OPTION_DTYPE)
    size_f, quality_f = options.dtype.names[:2]
    for j, (level, keep) in enumerate(forms):
        kept = np.maximum(1, (tokens * keep).astype(np.int64))
        options[size_f][j::len(forms)] = (kept // 256) * chunk[level][256] + chunk[level][kept % 256]
        options[quality_f][j::len(forms)] = np.maximum(0.0, (1 - sens_q * (level / 3.0) ** 2) * (1 - sens_d * ((1 - keep) / 0.875) ** 1.5))
    begin = np.arange(0, n * len(forms) + 1, len(forms), dtype=np.int32)
    capacity = int(options[size_f][0::len(forms)].sum() // 8)
    times = []
    for _ in range(max(1, min(args.steps or 3, 5))):
        t = time.perf_counter()
        choice, used, total = kvh.policy_assign(freq, options, begin, 2.0, 25e9, capacity)
        times.append(time.perf_counter() - t)
    assert used <= capacity
    print(json.dumps({"metric": "policy entries/s (host, one core)", "value": n / min(times), "unit": "entries/s", "entries": n,
                      "options_per_entry": len(forms), "seconds": round(min(times), 4), "us_per_entry": round(min(times) / n * 1e6, 3),
                      "capacity_bytes": capacity, "used_bytes": int(used), "stored_entries": int((choice >= 0).sum()),
                      "data": "synthetic"}))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def relaunch_as_ranks(n: int) -> int:
    """Start this script again as n ranks of one node (one process per GPU) and wait for them."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default: sized so the timed region stays short)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=WORKLOAD_NAMES, default="llama3-70b-32k")
    ap.add_argument("--variant", choices=["default", "static"], default="default",
                    help="library build: 'static' walks tiles with a fixed stride (scheduling comparison)")
    ap.add_argument("--tokens", type=int, default=0, help="shorten the context (profiling only; not a bench line)")
    ap.add_argument("--shape", default="", metavar="L,C,N",
                    help="a single context of L layers, C channels, N tokens instead of a named workload (other row widths)")
    ap.add_argument("--policy-entries", type=int, default=0,
                    help="time the policy (host code) on this many synthetic entries instead of the codec, and exit")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--stat-launches", type=int, default=50, help="launches per level and direction in level_stats; 0 skips")
    ap.add_argument("--extras-reps", type=int, default=20, help="launches per transcode pair / token-dropping level in extras")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the transcode / token-dropping / mix-ceiling timings")
    ap.add_argument("--print-source-digest", action="store_true", help="print kernel_source_digest() and exit")
    args = ap.parse_args()
    if args.print_source_digest:
        print(kernel_source_digest())
        return
    if args.policy_entries > 0:
        run_policy(args)
        return
    if args.shape:
        l, c, n = (int(x) for x in args.shape.split(","))
        name = f"custom-l{l}-c{c}-n{n}"
        SHAPES[name] = workloads.Shape(name, l, c, n)
        WORKLOAD_NAMES.append(name)
        args.workload = name
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(relaunch_as_ranks(args.gpus))
    if args.steps is None:
        # timed region of about half a second or more, so that the clock sampler sees it
        args.steps = {"tiny": 1000, "llama3-8b-8k": 300, BATCH: 20}.get(args.workload, 50)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.tokens and args.workload == BATCH:
        ap.error("--tokens applies to the single-context workloads")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
