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


def check_sampled_chunks(kvh, chunk_src, N, level_of_chunk, sample, streams, descs, table, pool, spare_pages):
    """chunk_src(i): the source tokens of chunk i, [l][2][n][c] on the GPU; streams/descs: what the
    GPU encoded; pool: what it decoded into."""
    ptable = table.cpu().numpy()

    def one(i):
        src = to_np16(chunk_src(i))
        l, _, n, c = src.shape
        assert n == min(256, N - 256 * i)
        level = level_of_chunk(i)
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
        check_sampled_chunks(kvh, lambda i: kv[:, :, 256 * i:min(N, 256 * i + 256)], N, lambda i: level, sample, streams,
                             descs, table, pool, perm[n_pages:].tolist())
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


def test_wide_rows_llama2_7b_shape(kvh):
    """32 KV heads x 128 = 4096 channels: the TMA-fed kernels work in column blocks of 1024."""
    s = workloads.LLAMA2_7B_4K
    run_context(kvh, s, seed=7000, levels=(0, 1, 2, 3), sample=[0, 15])


def test_batched_mixed_level_load_at_scale(kvh):
    """The batched mixed-level workload at its full size: 64 contexts of the 8B shape (32 layers),
    lengths log-uniform in [2K, 32K] with partial last chunks, a random level per chunk, one shared
    pool (~93 GB) behind one shuffled page table, ONE decode launch over ~2,800 chunks (~48 GB of
    streams).  On a GPU with less free memory the layer count is reduced to what fits; the launch
    geometry per layer stays the benchmark's."""
    c = 1024
    lengths = workloads.context_lengths(workloads.BATCH_N_CONTEXTS, workloads.BATCH_MIN_TOKENS,
                                        workloads.BATCH_MAX_TOKENS, seed=3000)
    assert len(lengths) == 64 and min(lengths) >= 2048 and max(lengths) <= 32768
    assert any(n % 256 for n in lengths)
    total_pages = sum(workloads.n_pages(n) for n in lengths)
    num_pages = total_pages + 100
    all_levels = [workloads.chunk_levels(workloads.n_chunks(N), 4, seed=3100 + i) for i, N in enumerate(lengths)]
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    per_layer = 2 * num_pages * 16 * c * 2                                   # pool
    per_layer += sum(kvh.plan_chunks(1, c, N, lv)[1] for N, lv in zip(lengths, all_levels))   # streams
    per_layer += 2 * 2 * max(lengths) * c * 2                                # one context's KV and slack
    l = int(max(1, min(32, (free - (12 << 30)) // per_layer)))
    if torch.cuda.get_device_properties(0).total_memory > (170 << 30):
        assert l == 32                                  # a 180 GB part runs the workload at its full size
    perm = workloads.shuffled_page_table(num_pages, num_pages, seed=3001)
    table = perm[:total_pages].cuda()
    pool = kvh.Pool.allocate(l, num_pages, c)
    pool.tensor.view(torch.int16).fill_(SENTINEL)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    plans, total_bytes, pt_base = [], 0, 0
    for i, N in enumerate(lengths):
        descs, size = kvh.plan_chunks(l, c, N, all_levels[i], stream_base=total_bytes, pt_base=pt_base)
        plans.append((N, all_levels[i], descs))
        total_bytes += size
        pt_base += workloads.n_pages(N)
    blob = torch.empty(total_bytes, dtype=torch.uint8, device="cuda")
    kept = {}                                          # (context, chunk) -> the chunk's source tokens
    for i, (N, levels, descs) in enumerate(plans):
        kv = workloads.make_kv(l, N, c, seed=3200 + i, device="cuda")
        local = descs.copy()
        base = int(descs["stream_off"][0])
        local["stream_off"] -= base
        size = int(local["stream_off"][-1]) + kvh.level_bytes(int(local["level"][-1]), l, c, int(local["n_tok"][-1]))
        kvh.encode_chunks(kv, kvh.descs_to_tensor(local, "cuda"), len(local), blob[base:base + size], status)
        if i in (0, 17, 63):
            last = len(levels) - 1
            for j in (0, last // 2, last):
                kept[(i, j)] = kv[:, :, 256 * j:min(N, 256 * j + 256)].clone()
        del kv
    all_descs = np.concatenate([d for _, _, d in plans])
    kvh.decode_batch(blob, kvh.descs_to_tensor(all_descs, "cuda"), len(all_descs), table, pool, status)
    assert status.item() == 0
    for i in (0, 17, 63):
        N, levels, descs = plans[i]
        sample = sorted(j for (ci, j) in kept if ci == i)
        check_sampled_chunks(kvh, lambda j: kept[(i, j)], N, lambda j: levels[j], sample, blob, descs, table, pool,
                             perm[total_pages:].tolist() if i == 0 else None)
