"""Parity at the sizes of the benchmark configurations, in the launch configuration bench.py
times (one kvh_encode and one kvh_decode_batch launch over the whole context).  The oracle
cannot run these sizes in full, so chunks are sampled: a sampled chunk's stream and its pages must
equal the oracle's bit for bit; pages nobody owns must keep their sentinel."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import SENTINEL, kvh, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu


def check_sampled_chunks(kvh, kv, level_of_chunk, sample, streams, descs, table, pool, spare_pages):
    """kv: [l][2][N][c] on the GPU; streams/descs: what the GPU encoded; pool: decoded into."""
    l, _, N, c = kv.shape
    ptable = table.cpu().numpy()

    def one(i):
        tok0 = 256 * i
        n = min(256, N - tok0)
        level = level_of_chunk(i)
        src = to_np16(kv[:, :, tok0:tok0 + n, :])
        want = oracle.encode_chunk(np.ascontiguousarray(src), 0, n, level)
        off = int(descs["stream_off"][i])
        got = streams[off:off + want.size].cpu().numpy()
        assert np.array_equal(got, want), f"stream of chunk {i} at level {level}"
        npg = -(-n // 16)
        ids = np.arange(npg, dtype=np.int32)
        ref = np.full(l * 2 * npg * 16 * c, SENTINEL, dtype=np.uint16)
        oracle.decode_chunk(want, level, l, c, n, ids, ref, 2 * npg * 16 * c, npg * 16 * c, 16 * c, npg)
        ref = ref.reshape(l, 2, npg, 16, c)
        pages = torch.from_numpy(ptable[int(descs["pt_off"][i]):int(descs["pt_off"][i]) + npg].astype(np.int64))
        have = to_np16(pool.tensor[:, :, pages.to(pool.tensor.device)])
        assert np.array_equal(have, ref), f"pages of chunk {i} at level {level}"

    with ThreadPoolExecutor(8) as ex:
        list(ex.map(one, sample))
    if spare_pages is not None and len(spare_pages):
        spare = to_np16(pool.tensor[:, :, torch.as_tensor(spare_pages, device=pool.tensor.device)])
        assert np.all(spare == SENTINEL)


def run_context(kvh, shape, seed, levels, sample):
    l, c, N = shape.n_layers, shape.n_channels, shape.n_tokens
    kv = workloads.make_kv(l, N, c, seed=seed, device="cuda")
    n_pages = workloads.n_pages(N)
    num_pages = n_pages + 64
    perm = workloads.shuffled_page_table(num_pages, num_pages, seed=seed)
    table = perm[:n_pages].cuda()
    pool = kvh.Pool.allocate(l, num_pages, c)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for level in levels:
        pool.tensor.view(torch.int16).fill_(SENTINEL)
        descs, total = kvh.plan_chunks(l, c, N, level)
        streams, used = kvh.encode(kv, level, dev_status=status)
        assert used == total
        kvh.decode_batch(streams, kvh.descs_to_tensor(descs, "cuda"), len(descs), table, pool, status)
        assert status.item() == 0
        check_sampled_chunks(kvh, kv, lambda i: level, sample, streams, descs, table, pool, perm[n_pages:].tolist())
        del streams


def test_llama8b_8k_every_level(kvh):
    s = workloads.LLAMA8B_8K
    run_context(kvh, s, seed=2000, levels=(0, 1, 2, 3), sample=[0, 13, 31])


def test_llama70b_32k_every_level(kvh):
    """The benchmark workload itself."""
    s = workloads.LLAMA70B_32K
    run_context(kvh, s, seed=4000, levels=(0, 1, 2, 3), sample=[0, 127])


def test_llama8b_128k_offsets_beyond_32_bits(kvh):
    """8.6e9 elements: element and byte offsets exceed 2^32 in the input, the stream and the pool."""
    s = workloads.LLAMA8B_128K
    run_context(kvh, s, seed=5000, levels=(0, 3), sample=[0, 300, 511])


def test_batched_mixed_level_load_at_scale(kvh):
    """64 contexts, lengths log-uniform in [2K, 32K] with partial last chunks, a random level per
    chunk, one shared pool behind one shuffled page table, ONE decode launch.  Eight layers
    instead of 32 keep the pool at ~23 GB; the launch geometry per layer is the benchmark's."""
    l, c = 8, 1024
    lengths = workloads.context_lengths(workloads.BATCH_N_CONTEXTS, workloads.BATCH_MIN_TOKENS,
                                        workloads.BATCH_MAX_TOKENS, seed=3000)
    assert len(lengths) == 64 and min(lengths) >= 2048 and max(lengths) <= 32768
    assert any(n % 256 for n in lengths)
    total_pages = sum(workloads.n_pages(n) for n in lengths)
    num_pages = total_pages + 100
    perm = workloads.shuffled_page_table(num_pages, num_pages, seed=3001)
    table = perm[:total_pages].cuda()
    pool = kvh.Pool.allocate(l, num_pages, c)
    pool.tensor.view(torch.int16).fill_(SENTINEL)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    plans, total_bytes, pt_base = [], 0, 0
    for i, N in enumerate(lengths):
        levels = workloads.chunk_levels(workloads.n_chunks(N), 4, seed=3100 + i)
        descs, size = kvh.plan_chunks(l, c, N, levels, stream_base=total_bytes, pt_base=pt_base)
        plans.append((N, levels, descs))
        total_bytes += size
        pt_base += workloads.n_pages(N)
    blob = torch.empty(total_bytes, dtype=torch.uint8, device="cuda")
    kept = {}
    for i, (N, levels, descs) in enumerate(plans):
        kv = workloads.make_kv(l, N, c, seed=3200 + i, device="cuda")
        local = descs.copy()
        base = int(descs["stream_off"][0])
        local["stream_off"] -= base
        size = int(local["stream_off"][-1]) + kvh.level_bytes(int(local["level"][-1]), l, c, int(local["n_tok"][-1]))
        kvh.encode_chunks(kv, kvh.descs_to_tensor(local, "cuda"), len(local), blob[base:base + size], status)
        if i in (0, 17, 63):
            kept[i] = kv
    all_descs = np.concatenate([d for _, _, d in plans])
    kvh.decode_batch(blob, kvh.descs_to_tensor(all_descs, "cuda"), len(all_descs), table, pool, status)
    assert status.item() == 0
    for i, kv in kept.items():
        N, levels, descs = plans[i]
        last = len(levels) - 1
        check_sampled_chunks(kvh, kv, lambda j: levels[j], [0, last // 2, last], blob, descs, table, pool,
                             perm[total_pages:].tolist() if i == 0 else None)
