#!/usr/bin/env python
"""Benchmark of the per-chunk KV-cache codec on the 70B-shaped context (l=80, c=1024, N=32768).

One step = one pass of the whole hot path over the context, for every level 0..3 in turn:
size arithmetic (host), encode of the context into its stored form, batched decode of all
chunks into a paged bf16 pool through a shuffled page table.  Inputs are resident in HBM when
the timed region starts.

  python bench.py [--gpus N] [--steps K] [--warmup W]            the CUDA library
  python bench.py --impl reference ...                           the CPU oracle, as it stands

Prints one JSON line (rank 0).  `value` is decode throughput in GB/s of bf16 written (the sum
over levels of bytes decoded over the sum of the decode intervals inside the timed steps);
`roofline` relates the decode kernel's algorithmic HBM bytes to the measured copy bandwidth;
`e2e` is the same metric with the stored form in pinned host memory (PCIe copy and status
read-back inside the timed interval); `cpu_baseline` times the oracle on the host cores.
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
from concurrent.futures import ThreadPoolExecutor

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
# DRAM traffic of one decode launch relative to its algorithmic bytes, from the ncu capture
# summarised in profiles/decode_tma_kernel_llama3-70b.md (dram__bytes_read + dram__bytes_write
# on a 4096-token slice of the same workload; traffic grows in proportion to the tokens).
DRAM_TRAFFIC_RATIO = {0: 0.981, 1: 0.973, 2: 0.967, 3: 0.964}
# the same for one encode launch (profiles/encode_tma_kernel_llama3-70b.md)
ENCODE_DRAM_TRAFFIC_RATIO = {0: 0.979, 1: 0.979, 2: 0.986, 3: 0.992}


def measured_peak() -> tuple[float, str]:
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(level: int, elements: int, stream_bytes: int) -> int:
    """Bytes one decode launch must move: the stored stream in, 2 bytes per element out."""
    return stream_bytes + 2 * elements


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines: list[str] = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
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
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


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


def oracle_inputs(shape: workloads.Shape, n_threads: int, target_s: float):
    """A slice of the workload (some layers, one chunk per thread) sized to about target_s per step."""
    import oracle
    oracle.build()
    probe = workloads.make_kv(1, 256 * n_threads, shape.n_channels, seed=4000)
    probe_np = probe.view(torch.int16).numpy().view(np.uint16)
    e, d, _ = oracle_sample_step(probe_np, n_threads)
    layers = max(1, min(shape.n_layers, int(target_s / max(e + d, 1e-3))))
    kv = workloads.make_kv(layers, 256 * n_threads, shape.n_channels, seed=4000)
    return kv.view(torch.int16).numpy().view(np.uint16), layers


def run_reference(args, shape: workloads.Shape):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return                                           # one CPU program: rank 0 alone runs it
    cores = len(os.sched_getaffinity(0))
    kv_np, layers = oracle_inputs(shape, cores, target_s=1.5)
    for _ in range(args.warmup):
        oracle_sample_step(kv_np, cores)
    enc = dec = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e, d, elements = oracle_sample_step(kv_np, cores)
        enc += e; dec += d
    total = time.perf_counter() - t0
    value = len(LEVELS) * 2 * elements * args.steps / dec / 1e9
    sample = f"{layers} of {shape.n_layers} layers x {cores} chunks of 256 tokens, every level, per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": shape.name, "n_layers": shape.n_layers, "n_channels": shape.n_channels,
                   "n_tokens": shape.n_tokens, "levels": list(LEVELS), "sample": sample},
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


def time_extras(kvh, kv, plans, stream_buf, status, l, c, N, n_chunks, dev, reps: int = 5):
    """Transcoding (every pair of levels) and token dropping (4 sink tokens + a recent window, a
    quarter of the context kept), each as the mean of `reps` launches over the whole context after
    one warm-up launch.  Bytes counted: streams read + streams written (transcode), kept bf16 rows
    read + streams written (token dropping)."""
    def timed(fn):
        fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        b.synchronize()
        return a.elapsed_time(b) / reps

    elements = l * 2 * N * c
    out = {"transcode": [], "token_dropping": []}
    second = torch.empty(plans[1][2], dtype=torch.uint8, device=dev)
    for lin in (0, 1, 2):
        _, descs_in_dev, total_in = plans[lin]
        kvh.encode(kv, lin, out=stream_buf[:total_in], dev_status=status)
        for lout in range(lin + 1, 4):
            _, descs_out_dev, total_out = plans[lout]
            ms = timed(lambda: kvh.transcode(stream_buf[:total_in], descs_in_dev, second[:total_out], descs_out_dev,
                                             n_chunks, l, c, lin, lout, dev_status=status))
            out["transcode"].append({"from": lin, "to": lout, "ms": round(ms, 4),
                                     "hbm_gbps": round((total_in + total_out) / ms / 1e6, 1),
                                     "tokens_per_s": round(N / ms * 1e3)})
    runs, n_kept = kvh.keep_sinks_and_recent(N, 4, N // 4 - 4)
    for level in LEVELS:
        descs, total = kvh.plan_chunks(l, c, n_kept, level)
        ms = timed(lambda: kvh.encode_kept(kv, runs, None, len(descs), second[:total], status, level=level))
        out["token_dropping"].append({"level": level, "kept_tokens": n_kept, "ms": round(ms, 4),
                                      "hbm_gbps": round((2 * elements * n_kept // N + total) / ms / 1e6, 1)})
    assert status.item() == 0
    return out


def run_ours(args, shape: workloads.Shape):
    import torch.distributed as dist
    import paper_2509_00105_b200 as kvh

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    kvh.lib()                                            # fails loudly if the extension is missing

    l, c, N = shape.n_layers, shape.n_channels, shape.n_tokens
    elements = l * 2 * N * c
    n_chunks = workloads.n_chunks(N)
    n_pages = workloads.n_pages(N)
    kv = workloads.make_kv(l, N, c, seed=rank_seed(rank), device=dev)   # every rank its own context
    pool = kvh.Pool.allocate(l, n_pages, c, device=dev)
    table = workloads.shuffled_page_table(n_pages, n_pages, seed=rank_seed(rank)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    plans = {}
    for level in LEVELS:
        descs, total = kvh.plan_chunks(l, c, N, level)
        assert total == sum(kvh.level_bytes(level, l, c, int(n)) for n in descs["n_tok"])
        plans[level] = (descs, kvh.descs_to_tensor(descs, dev), total)
    stream_buf = torch.empty(max(p[2] for p in plans.values()), dtype=torch.uint8, device=dev)

    def step(events=None):
        for level in LEVELS:
            descs, descs_dev, total = plans[level]
            if events is not None:
                events[level][0].record()
            kvh.encode(kv, level, out=stream_buf[:total], dev_status=status)
            if events is not None:
                events[level][1].record()
            kvh.decode_batch(stream_buf[:total], descs_dev, n_chunks, table, pool, status)
            if events is not None:
                events[level][2].record()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 0)):
        step()
    ev = [{lv: [torch.cuda.Event(enable_timing=True) for _ in range(3)] for lv in LEVELS} for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    t_start.record()
    for s in range(args.steps):
        step(ev[s])
    t_end.record()
    barrier()
    clocks = sampler.stop()
    assert status.item() == 0, f"device status {status.item()}"

    total_ms = t_start.elapsed_time(t_end)
    enc_ms = {lv: sum(e[lv][0].elapsed_time(e[lv][1]) for e in ev) / args.steps for lv in LEVELS}
    dec_ms = {lv: sum(e[lv][1].elapsed_time(e[lv][2]) for e in ev) / args.steps for lv in LEVELS}
    # spread of the per-launch times on this rank (the means above are what the metric uses)
    dec_all = {lv: sorted(e[lv][1].elapsed_time(e[lv][2]) for e in ev) for lv in LEVELS}
    enc_all = {lv: sorted(e[lv][0].elapsed_time(e[lv][1]) for e in ev) for lv in LEVELS}
    times = max_over_ranks([total_ms] + [enc_ms[lv] for lv in LEVELS] + [dec_ms[lv] for lv in LEVELS], dev, world)
    total_ms = times[0]
    enc_ms = dict(zip(LEVELS, times[1:5]))
    dec_ms = dict(zip(LEVELS, times[5:9]))

    # ---- the two further store-side operations, timed on their own after the steps ----
    extras = None
    if world == 1 and not args.no_extras:
        extras = time_extras(kvh, kv, plans, stream_buf, status, l, c, N, n_chunks, dev)

    # ---- end to end: stored form in pinned host memory ----
    e2e = None
    if not args.no_e2e:
        host = torch.empty(stream_buf.numel(), dtype=torch.uint8).pin_memory()
        host_status = torch.zeros(1, dtype=torch.int32).pin_memory()
        copy_stream = torch.cuda.Stream(device=dev)
        main_stream = torch.cuda.Stream(device=dev)
        k_e2e = max(1, min(args.steps, args.e2e_steps))
        load_ms = {lv: 0.0 for lv in LEVELS}
        store_ms = {lv: 0.0 for lv in LEVELS}
        with torch.cuda.stream(main_stream):
            for it in range(1 + k_e2e):                  # one untimed pass first
                for level in LEVELS:
                    descs, descs_dev, total = plans[level]
                    a, b, d = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                    a.record()
                    kvh.store_host(kv, descs, descs_dev, stream_buf, host, status, host_status, copy_stream)
                    b.record()
                    kvh.load_host(host, stream_buf, descs, descs_dev, table, pool, status, host_status, copy_stream)
                    d.record()
                    d.synchronize()
                    assert host_status.item() == 0
                    if it > 0:
                        store_ms[level] += a.elapsed_time(b) / k_e2e
                        load_ms[level] += b.elapsed_time(d) / k_e2e
        t = max_over_ranks([load_ms[lv] for lv in LEVELS] + [store_ms[lv] for lv in LEVELS], dev, world)
        load_ms, store_ms = dict(zip(LEVELS, t[:4])), dict(zip(LEVELS, t[4:]))
        stream_total = sum(plans[lv][2] for lv in LEVELS)
        e2e = {"value": whole_job_gbps(world, len(LEVELS) * 2 * elements, sum(load_ms.values())), "unit": UNIT,
               "h2d_bytes_per_step": stream_total, "d2h_bytes_per_step": stream_total + 4 * 2 * len(LEVELS),
               "steps": k_e2e, "what": "kvh_load_host: pinned host streams -> HBM -> pages, status read back",
               "load_ms_per_level": [round(load_ms[lv], 3) for lv in LEVELS],
               "store_ms_per_level": [round(store_ms[lv], 3) for lv in LEVELS],
               "store_gbps_bf16_in": whole_job_gbps(world, len(LEVELS) * 2 * elements, sum(store_ms.values()))}
        del host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    levels_out = []
    for lv in LEVELS:
        alg = algorithmic_bytes(lv, elements, plans[lv][2])
        levels_out.append({
            "level": lv, "bits": CODE_BITS[lv], "stream_bytes": plans[lv][2],
            "decode_ms": round(dec_ms[lv], 4), "decode_ms_median": round(statistics.median(dec_all[lv]), 4),
            "decode_ms_min": round(dec_all[lv][0], 4), "encode_ms_median": round(statistics.median(enc_all[lv]), 4),
            "encode_ms_min": round(enc_all[lv][0], 4), "decode_gbps_bf16_out": round(2 * elements / dec_ms[lv] / 1e6, 1),
            "decode_hbm_gbps": round(alg / dec_ms[lv] / 1e6, 1), "decode_roofline_frac": round(alg / dec_ms[lv] / 1e6 / peak, 4),
            "decode_tokens_per_s": round(N / dec_ms[lv] * 1e3), "encode_ms": round(enc_ms[lv], 4),
            "encode_hbm_gbps": round(alg / enc_ms[lv] / 1e6, 1), "encode_roofline_frac": round(alg / enc_ms[lv] / 1e6 / peak, 4)})
    dec_total_ms = sum(dec_ms.values())
    alg_total = sum(algorithmic_bytes(lv, elements, plans[lv][2]) for lv in LEVELS)
    achieved = alg_total / dec_total_ms / 1e6
    ratios = [DRAM_TRAFFIC_RATIO[lv] for lv in LEVELS]
    traffic = None
    if all(r is not None for r in ratios):
        traffic = sum(r * algorithmic_bytes(lv, elements, plans[lv][2]) for r, lv in zip(ratios, LEVELS)) / len(LEVELS)
    out = {
        "metric": METRIC, "value": whole_job_gbps(world, len(LEVELS) * 2 * elements, dec_total_ms), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": shape.name, "n_layers": l, "n_channels": c, "n_tokens": N, "chunk_tokens": 256,
                   "page_tokens": 16, "levels": list(LEVELS), "step": "encode + batched decode-to-pages at every level",
                   "l2": "inputs larger than L2 (10.7 GB KV, 10.7 GB pool per rank)", "parallelism": f"replicas x{world}"},
        "decode_ms_per_step": dec_total_ms, "encode_ms_per_step": sum(enc_ms.values()),
        "tokens_per_s_loaded": world * len(LEVELS) * N / dec_total_ms * 1e3,
        "levels": levels_out,
        "roofline": {"bound": "hbm", "kernel": "decode_tma_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                     "frac_of_8TBs_datasheet": achieved / 8000.0,
                     "per_launch": "mean over the 4 launches of a step (one per level): stream bytes + 2 B/element"},
        "roofline_encode": {"bound": "hbm", "kernel": "encode_tma_kernel", "achieved": alg_total / sum(enc_ms.values()) / 1e6,
                            "peak": peak, "unit": "GB/s", "frac": alg_total / sum(enc_ms.values()) / 1e6 / peak,
                            "traffic": sum(ENCODE_DRAM_TRAFFIC_RATIO[lv] * algorithmic_bytes(lv, elements, plans[lv][2])
                                           for lv in LEVELS) / len(LEVELS),
                            "peak_kind": f"of {peak_kind}",
                            "per_launch": "mean over the 4 launches of a step: 2 B/element + stream bytes"},
        "gpu_launches": args.steps * 2 * len(LEVELS),
        "clocks": clocks,
    }
    if e2e is not None:
        out["e2e"] = e2e
    if extras is not None:
        for rows in extras.values():
            for r in rows:
                r["roofline_frac"] = round(r["hbm_gbps"] / peak, 4)
        out["extras"] = extras
    if world == 1 and not args.no_cpu_baseline:
        cores = len(os.sched_getaffinity(0))
        kv_np, layers = oracle_inputs(shape, cores, target_s=4.0)
        e, d, el = oracle_sample_step(kv_np, cores)
        one_np = np.ascontiguousarray(kv_np[:max(1, kv_np.shape[0] // 8), :, :256])     # one chunk, an eighth of the layers
        e1, d1, el1 = oracle_sample_step(one_np, 1)
        out["cpu_baseline"] = {
            "single_thread_value": len(LEVELS) * 2 * el1 / d1 / 1e9,
            "value": len(LEVELS) * 2 * el / d / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{layers} of {l} layers x {cores} chunks of 256 tokens, every level, encode {e:.1f} s + decode {d:.1f} s",
            "encode_gbps_bf16_in": len(LEVELS) * 2 * el / e / 1e9}
        # the sample's rates applied to the whole step (every level of the full context): not measured
        full = len(LEVELS) * 2.0 * l * 2 * N * c
        out["cpu_baseline"]["extrapolated_step_s"] = round(full / (len(LEVELS) * 2 * el) * (e + d), 1)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--tokens", type=int, default=0, help="shorten the context (profiling only; not a bench line)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the transcode / token-dropping timings")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    shape = workloads.LLAMA70B_32K
    if args.tokens:
        shape = workloads.Shape(f"{shape.name}-first{args.tokens}", shape.n_layers, shape.n_channels, args.tokens)
    if args.impl == "reference":
        run_reference(args, shape)
    else:
        run_ours(args, shape)


if __name__ == "__main__":
    main()
