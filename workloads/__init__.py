"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds none of the codec's arithmetic: it only draws KV tensors,
context lengths, per-chunk levels and page tables.  The paper evaluates on
LongBench contexts run through Llama-3.1-8B-Instruct; neither the datasets nor
the weights are available here, so these inputs stand in for them and take only
the KV *shapes* of the Llama-3 8B / 70B models (8 KV heads x 128 channels, 32 or
80 layers) and a value distribution with per-channel scale spread and a few
large-magnitude K channels.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

CHUNK_TOKENS = 256
PAGE_TOKENS = 16
PAGES_PER_CHUNK = CHUNK_TOKENS // PAGE_TOKENS


@dataclass(frozen=True)
class Shape:
    name: str
    n_layers: int
    n_channels: int
    n_tokens: int


# The shapes of the five benchmark workloads.
TINY = Shape("tiny", 4, 1024, 256)
LLAMA8B_8K = Shape("llama3-8b-8k", 32, 1024, 8192)
LLAMA70B_32K = Shape("llama3-70b-32k", 80, 1024, 32768)
LLAMA8B_128K = Shape("llama3-8b-128k", 32, 1024, 131072)
# a multi-head model without grouped KV heads (32 heads x 128): rows wider than the 1024 of the Llama-3 shapes
LLAMA2_7B_4K = Shape("llama2-7b-4k", 32, 4096, 4096)
BATCH_N_CONTEXTS = 64
BATCH_MIN_TOKENS = 2048
BATCH_MAX_TOKENS = 32768


def make_kv(n_layers: int, n_tokens: int, n_channels: int, seed: int, device="cpu",
            outlier_frac: float = 0.01, outlier_gain: float = 10.0) -> torch.Tensor:
    """bf16 tensor [l][2][N][c]: N(0,1) times a per-(layer, K/V, channel) scale
    drawn from lognormal(0, 0.5); for K only, round(outlier_frac * c) channels
    per layer are multiplied by outlier_gain.  Deterministic per (seed, device
    type); CPU and CUDA streams differ, which is fine because each consumer
    hands the same tensor to both sides."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    out = torch.empty((n_layers, 2, n_tokens, n_channels), dtype=torch.bfloat16, device=dev)
    n_out = int(round(outlier_frac * n_channels))
    for layer in range(n_layers):
        for kv in range(2):
            s = torch.exp(0.5 * torch.randn(n_channels, generator=g, device=dev))
            if kv == 0 and n_out > 0:
                idx = torch.randperm(n_channels, generator=g, device=dev)[:n_out]
                s[idx] *= outlier_gain
            # token blocks bound the fp32 temporary for long contexts
            for t0 in range(0, n_tokens, 8192):
                t1 = min(n_tokens, t0 + 8192)
                x = torch.randn((t1 - t0, n_channels), generator=g, device=dev)
                out[layer, kv, t0:t1] = (x * s).to(torch.bfloat16)
    return out


def context_lengths(n_contexts: int, lo: int, hi: int, seed: int) -> list[int]:
    """Lengths log-uniform in [lo, hi] tokens (partial last chunks allowed)."""
    g = torch.Generator().manual_seed(seed)
    u = torch.rand(n_contexts, generator=g, dtype=torch.float64)
    return [int(round(math.exp(math.log(lo) + float(x) * (math.log(hi) - math.log(lo))))) for x in u]


def chunk_levels(n_chunks: int, n_levels: int, seed: int) -> list[int]:
    """One uniformly random level per chunk."""
    g = torch.Generator().manual_seed(seed)
    return torch.randint(0, n_levels, (n_chunks,), generator=g).tolist()


def shuffled_page_table(n_pages_needed: int, n_pages_pool: int, seed: int) -> torch.Tensor:
    """int32 page ids: the first n_pages_needed entries of a seeded permutation
    of the pool's pages (distinct, scattered)."""
    assert n_pages_needed <= n_pages_pool
    g = torch.Generator().manual_seed(seed)
    return torch.randperm(n_pages_pool, generator=g)[:n_pages_needed].to(torch.int32)


def n_chunks(n_tokens: int) -> int:
    return (n_tokens + CHUNK_TOKENS - 1) // CHUNK_TOKENS


def n_pages(n_tokens: int) -> int:
    """Pages a context occupies; chunk i of a context starts at page slot 16*i."""
    return (n_tokens + PAGE_TOKENS - 1) // PAGE_TOKENS


def policy_entries(n_entries: int, seed: int):
    """Synthetic inputs of the policy: per entry a reuse frequency (Zipf-like), a length in tokens
    (log-uniform in [2K, 32K]) and, for every stored form on offer, an estimated quality.  Stored
    forms: quantisation level 0..3 crossed with the kept fraction of tokens (1, 1/2, 1/4, 1/8).
    Quality falls with coarser levels and with dropped tokens, each entry with its own sensitivity
    (some texts tolerate dropping, others quantisation); the numbers stand in for the profiled
    quality curves the paper's estimator measures with a language model, which is not available
    here.  Returns (freq [n], n_tokens [n], forms [(level, keep_fraction)], quality [n][len(forms)])."""
    g = torch.Generator().manual_seed(seed)
    rank = torch.randperm(n_entries, generator=g).to(torch.float64) + 1.0
    freq = (10.0 / rank).tolist()
    tokens = context_lengths(n_entries, BATCH_MIN_TOKENS, BATCH_MAX_TOKENS, seed + 1)
    forms = [(level, keep) for keep in (1.0, 0.5, 0.25, 0.125) for level in range(4)]
    sens_q = 0.02 + 0.25 * torch.rand(n_entries, generator=g, dtype=torch.float64)     # loss at 2 bits
    sens_d = 0.05 + 0.9 * torch.rand(n_entries, generator=g, dtype=torch.float64)      # loss when all but 1/8 is dropped
    quality = []
    for i in range(n_entries):
        row = []
        for level, keep in forms:
            loss_q = float(sens_q[i]) * (level / 3.0) ** 2
            loss_d = float(sens_d[i]) * ((1.0 - keep) / 0.875) ** 1.5
            row.append(max(0.0, (1.0 - loss_q) * (1.0 - loss_d)))
        quality.append(row)
    return freq, tokens, forms, quality
