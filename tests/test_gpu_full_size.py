"""Parity at the sizes of the five benchmark configurations, in the launch configuration bench.py
times (one kvh_encode and one kvh_decode_batch launch over the whole context), at every level.

Three kinds of evidence, because the oracle cannot run the largest sizes in full:
  * against the oracle, bit for bit: every chunk of the 8K context, and chunks spread over the whole
    launch (first, last, middle and one in about eight in between) of the larger ones: a sampled
    chunk's stream and its pages must equal the oracle's;
  * whole buffers, every byte: the complete stream and the complete pool of the library proper (the
    persistent TMA-fed kernels, tiles handed out dynamically) must equal those of the "direct" build
    (one CTA per tile, plain loads), two independent implementations; and a second run of the same
    decode must reproduce the pool, since which CTA takes which tile changes from run to run;
  * coverage: every page the table names is written in full, pages nobody owns keep their sentinel.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import SENTINEL, kvh, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu

CORES = len(os.sched_getaffinity(0))


def spread(n_chunks, step):
    """First, last, the two middle chunks and one in every `step` in between."""
    return sorted(set([0, n_chunks - 1, n_chunks // 2 - 1, n_chunks // 2] + list(range(step // 2, n_chunks, step))))


def check_sampled_chunks(kvh, chunk_src, N, level_of_chunk, sample, streams, descs, table, pool, spare_pages):
    """chunk_src(i): the source tokens of chunk i, [l][2][n][c] on the GPU; streams/descs: what the
    GPU encoded; pool: what it decoded into."""
    ptable = table.cpu().numpy()

    def fetch(i):                                       # device reads stay on this thread
        src = to_np16(chunk_src(i))
        l, _, n, c = src.shape
        level = level_of_chunk(i)
        off = int(descs["stream_off"][i])
        size = oracle.level_bytes(level, l, c, n)
        got = streams[off:off + size].cpu().numpy()
        npg = -(-n // 16)
        pages = torch.from_numpy(ptable[int(descs["pt_off"][i]):int(descs["pt_off"][i]) + npg].astype(np.int64))
        have = to_np16(pool.tensor[:, :, pages.to(pool.tensor.device)])
        return i, src, level, got, have

    def one(args):                                      # the oracle's part: ctypes releases the GIL
        i, src, level, got, have = args
        l, _, n, c = src.shape
        assert n == min(256, N - 256 * i)
        want = oracle.encode_chunk(np.ascontiguousarray(src), 0, n, level)
        assert np.array_equal(got, want), f"stream of chunk {i} at level {level}"
        npg = -(-n // 16)
        ids = np.arange(npg, dtype=np.int32)
        ref = np.full(l * 2 * npg * 16 * c, SENTINEL, dtype=np.uint16)
        oracle.decode_chunk(want, level, l, c, n, ids, ref, 2 * npg * 16 * c, npg * 16 * c, 16 * c, npg)
        assert np.array_equal(have, ref.reshape(l, 2, npg, 16, c)), f"pages of chunk {i} at level {level}"

    with ThreadPoolExecutor(CORES) as ex:
        futures = [ex.submit(one, fetch(i)) for i in sample]
        for f in futures:
            f.result()
    if spare_pages is not None and len(spare_pages):
        spare = to_np16(pool.tensor[:, :, torch.as_tensor(spare_pages, device=pool.tensor.device)])
        assert np.all(spare == SENTINEL)


def assert_every_owned_row_written(pool, table):
    """No sentinel is left in any page the table names (the contexts checked this way end on a page
    boundary).  Layer by layer, to bound the temporary."""
    idx = table.long()
    sentinel = SENTINEL                                  # 0x7FC1 is positive as a signed 16-bit value
    for layer in range(pool.tensor.shape[0]):
        pages = pool.tensor[layer][:, idx].view(torch.int16)
        assert not bool((pages == sentinel).any()), f"unwritten row in layer {layer}"


def run_context(kvh, shape, seed, levels, sample):
    direct = kvh.variant("direct")
    l, c, N = shape.n_layers, shape.n_channels, shape.n_tokens
    assert N % 16 == 0
    kv = workloads.make_kv(l, N, c, seed=seed, device="cuda")
    n_pages = workloads.n_pages(N)
    num_pages = n_pages + 64
    perm = workloads.shuffled_page_table(num_pages, num_pages, seed=seed)
    table = perm[:n_pages].cuda()
    pool = kvh.Pool.allocate(l, num_pages, c)
    pool_b = direct.Pool.allocate(l, num_pages, c)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for level in levels:
        pool.tensor.view(torch.int16).fill_(SENTINEL)
        pool_b.tensor.view(torch.int16).fill_(SENTINEL)
        descs, total = kvh.plan_chunks(l, c, N, level)
        descs_dev = kvh.descs_to_tensor(descs, "cuda")
        streams, used = kvh.encode(kv, level, dev_status=status)
        assert used == total
        kvh.decode_batch(streams, descs_dev, len(descs), table, pool, status)
        assert status.item() == 0
        # the oracle on the sampled chunks
        check_sampled_chunks(kvh, lambda i: kv[:, :, 256 * i:min(N, 256 * i + 256)], N, lambda i: level, sample, streams,
                             descs, table, pool, perm[n_pages:].tolist())
        assert_every_owned_row_written(pool, table)
        # the other kernel family on every byte
        streams_b, _ = direct.encode(kv, level, dev_status=status)
        assert torch.equal(streams, streams_b), f"TMA-fed and direct encoders differ at level {level}"
        del streams_b
        direct.decode_batch(streams, descs_dev, len(descs), table, pool_b, status)
        assert status.item() == 0
        assert torch.equal(pool.tensor.view(torch.int16), pool_b.tensor.view(torch.int16)), \
            f"TMA-fed and direct decoders differ at level {level}"
        # the same launch again: the dynamic hand-out of tiles must not change a byte
        pool.tensor.view(torch.int16).fill_(SENTINEL)
        kvh.decode_batch(streams, descs_dev, len(descs), table, pool, status)
        streams_again, _ = kvh.encode(kv, level, dev_status=status)
        assert status.item() == 0
        assert torch.equal(pool.tensor.view(torch.int16), pool_b.tensor.view(torch.int16))
        assert torch.equal(streams, streams_again)
        del streams, streams_again


def test_tiny_single_context_every_level(kvh):
    s = workloads.TINY
    run_context(kvh, s, seed=0, levels=(0, 1, 2, 3), sample=[0])


def test_llama8b_8k_every_level_every_chunk(kvh):
    s = workloads.LLAMA8B_8K
    run_context(kvh, s, seed=2000, levels=(0, 1, 2, 3), sample=list(range(workloads.n_chunks(s.n_tokens))))


def test_llama70b_32k_every_level(kvh):
    """The benchmark workload itself: 17 of its 128 chunks against the oracle, all of it against the
    other kernel family."""
    s = workloads.LLAMA70B_32K
    run_context(kvh, s, seed=4000, levels=(0, 1, 2, 3), sample=spread(workloads.n_chunks(s.n_tokens), 8))


def test_llama8b_128k_offsets_beyond_32_bits(kvh):
    """8.6e9 elements: element and byte offsets exceed 2^32 in the input, the stream and the pool, at
    every level."""
    s = workloads.LLAMA8B_128K
    run_context(kvh, s, seed=5000, levels=(0, 1, 2, 3), sample=spread(workloads.n_chunks(s.n_tokens), 32))


def test_wide_rows_llama2_7b_shape(kvh):
    """32 KV heads x 128 = 4096 channels: the TMA-fed kernels work in column blocks of 1024."""
    s = workloads.LLAMA2_7B_4K
    run_context(kvh, s, seed=7000, levels=(0, 1, 2, 3), sample=[0, 7, 15])


@pytest.mark.parametrize("c", [256, 768, 1280])
def test_other_row_widths_at_scale(kvh, c):
    """Rows that are not 1024 channels wide take other routes through the same kernels: 2 KV heads
    (256 channels: four tiles per work unit), 6 heads (768: the general consumers, 2-D boxes in the
    encoder) and 10 heads (1280: two column blocks of 640, one copy per row).  16 layers x 16,384
    tokens each: thousands of units per launch, dynamic hand-out, every level; sampled chunks against
    the oracle and whole buffers against the other kernel family."""
    s = workloads.Shape(f"rows-{c}", 16, c, 16384)
    run_context(kvh, s, seed=7100 + c, levels=(0, 1, 2, 3), sample=spread(workloads.n_chunks(s.n_tokens), 16))


def plane_checksums(pool):
    """Two position-dependent 64-bit sums per (layer, K|V) plane (wrap-around arithmetic)."""
    out = []
    w = None
    for layer in range(pool.tensor.shape[0]):
        for kv in range(2):
            v = pool.tensor[layer, kv].reshape(-1).view(torch.int32).to(torch.int64)
            if w is None:
                w = (torch.arange(v.numel(), device=v.device, dtype=torch.int64) % 65521) + 1
            out.append((int(v.sum()), int((v * w).sum())))
            del v
    return out


def test_batched_mixed_level_load_at_scale(kvh):
    """The batched mixed-level workload at its full size: 64 contexts of the 8B shape (32 layers),
    lengths log-uniform in [2K, 32K] with partial last chunks, a random level per chunk, one shared
    pool (~93 GB) behind one shuffled page table, ONE decode launch over ~2,800 chunks (~48 GB of
    streams).  On a GPU with less free memory the layer count is reduced to what fits; the launch
    geometry per layer stays the benchmark's.  Two pools of this size do not fit side by side, so
    the other kernel family and the repeated launch are compared through per-plane checksums."""
    direct = kvh.variant("direct")
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
    l = int(max(1, min(32, (free - (16 << 30)) // per_layer)))
    if torch.cuda.get_device_properties(0).total_memory > (170 << 30):
        assert l == 32                                  # a 180 GB part runs the workload at its full size
    perm = workloads.shuffled_page_table(num_pages, num_pages, seed=3001)
    table = perm[:total_pages].cuda()
    pool = kvh.Pool.allocate(l, num_pages, c)
    pool.tensor.view(torch.int16).fill_(SENTINEL)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    sampled_contexts = (0, 9, 17, 31, 45, 63)
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
        if i in sampled_contexts:
            last = len(levels) - 1
            for j in sorted({0, last // 3, 2 * last // 3, last}):
                kept[(i, j)] = kv[:, :, 256 * j:min(N, 256 * j + 256)].clone()
        del kv
    all_descs = np.concatenate([d for _, _, d in plans])
    all_descs_dev = kvh.descs_to_tensor(all_descs, "cuda")
    kvh.decode_batch(blob, all_descs_dev, len(all_descs), table, pool, status)
    assert status.item() == 0
    assert {lv for _, levels, _ in plans for lv in levels} == {0, 1, 2, 3}
    for i in sampled_contexts:
        N, levels, descs = plans[i]
        sample = sorted(j for (ci, j) in kept if ci == i)
        check_sampled_chunks(kvh, lambda j: kept[(i, j)], N, lambda j: levels[j], sample, blob, descs, table, pool,
                             perm[total_pages:].tolist() if i == 0 else None)
    kept.clear()
    sums = plane_checksums(pool)
    # the same launch again, then the other kernel family: every plane of the pool must come out the same
    pool.tensor.view(torch.int16).fill_(SENTINEL)
    kvh.decode_batch(blob, all_descs_dev, len(all_descs), table, pool, status)
    assert plane_checksums(pool) == sums
    pool.tensor.view(torch.int16).fill_(SENTINEL)
    direct.decode_batch(blob, all_descs_dev, len(all_descs), table, direct.Pool(pool.tensor), status)
    assert status.item() == 0
    assert plane_checksums(pool) == sums


def test_transcode_at_full_size_equals_decode_then_encode(kvh):
    """The benchmark's transcoding launches (70B shape, 32,768 tokens), every pair of levels, whole
    buffers: transcoding a stored context must give, byte for byte, what encoding at the new level
    gives from the pages the old stream decodes to (the definition of the operation; both of those
    paths are checked against the oracle above), and chunks spread over the launch must equal the
    oracle's transcoding of the same stored bytes."""
    s = workloads.LLAMA70B_32K
    l, c, N = s.n_layers, s.n_channels, s.n_tokens
    kv = workloads.make_kv(l, N, c, seed=4100, device="cuda")
    n_pages = workloads.n_pages(N)
    table = torch.arange(n_pages, dtype=torch.int32, device="cuda")          # identity: the pool is laid out like kv
    pool = kvh.Pool.allocate(l, n_pages, c)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plans = {k: kvh.plan_chunks(l, c, N, k) for k in range(4)}
    devs = {k: kvh.descs_to_tensor(plans[k][0], "cuda") for k in range(4)}
    n_chunks = len(plans[0][0])
    sample = spread(n_chunks, 32)
    for lin in (0, 1, 2):
        src, _ = kvh.encode(kv, lin, dev_status=status)
        pool.tensor.view(torch.int16).fill_(SENTINEL)
        kvh.decode_batch(src, devs[lin], n_chunks, table, pool, status)
        decoded = pool.tensor.view(l, 2, N, c)
        for lout in range(lin + 1, 4):
            want, total = kvh.encode(decoded, lout, dev_status=status)
            got = torch.full((total + 256,), 0xAB, dtype=torch.uint8, device="cuda")
            kvh.transcode(src, devs[lin], got[:total], devs[lout], n_chunks, l, c, lin, lout, dev_status=status)
            assert status.item() == 0
            assert torch.equal(got[:total], want), f"transcode {lin}->{lout} differs from decode + encode"
            assert bool((got[total:] == 0xAB).all())
            if lin > 0:                                  # from level 0 the operation is the encoder itself

                def one(i):
                    a, b = int(plans[lin][0]["stream_off"][i]), int(plans[lout][0]["stream_off"][i])
                    size_in = oracle.level_bytes(lin, l, c, 256)
                    size_out = oracle.level_bytes(lout, l, c, 256)
                    ref = oracle.transcode_chunk(src[a:a + size_in].cpu().numpy(), lin, lout, l, c, 256)
                    assert np.array_equal(got[b:b + size_out].cpu().numpy(), ref), f"chunk {i}, {lin}->{lout}"

                for i in sample[::3]:
                    one(i)
            del want, got
        del src


def test_token_dropping_at_full_size(kvh):
    """The benchmark's token-dropping launches (70B shape, 4 sink tokens and a recent window, a quarter
    of the context kept) at every level, whole buffers: encoding the kept runs must give, byte for
    byte, the encoding of the compacted tensor (the definition of the operation)."""
    s = workloads.LLAMA70B_32K
    l, c, N = s.n_layers, s.n_channels, s.n_tokens
    kv = workloads.make_kv(l, N, c, seed=4200, device="cuda")
    runs, n_kept = kvh.keep_sinks_and_recent(N, 4, N // 4 - 4)
    assert n_kept == N // 4 and len(runs) == 2
    compact = torch.cat([kv[:, :, int(r["first"]):int(r["first"]) + int(r["count"])] for r in runs], dim=2).contiguous()
    assert compact.shape[2] == n_kept
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for level in (0, 1, 2, 3):
        want, total = kvh.encode(compact, level, dev_status=status)
        got = torch.full((total + 256,), 0xAB, dtype=torch.uint8, device="cuda")
        kvh.encode_kept(kv, runs, None, workloads.n_chunks(n_kept), got[:total], status, level=level)
        assert status.item() == 0
        assert torch.equal(got[:total], want), f"kept-run encoding differs from the compacted encoding at level {level}"
        assert bool((got[total:] == 0xAB).all())


def test_host_tier_at_full_size_with_a_level_per_chunk(kvh):
    """The benchmark's end-to-end path at its full size (70B shape, 32,768 tokens), here with a random
    level per chunk so that slices mix levels: what kvh_store_host leaves in pinned host memory must be,
    byte for byte, what kvh_encode_chunks writes on the device, and what kvh_load_host decodes from
    there must be, element for element, what one batched decode of the device copy gives (both of
    those are checked against the oracle above)."""
    s = workloads.LLAMA70B_32K
    l, c, N = s.n_layers, s.n_channels, s.n_tokens
    kv = workloads.make_kv(l, N, c, seed=4300, device="cuda")
    levels = workloads.chunk_levels(workloads.n_chunks(N), 4, seed=4301)
    descs, total = kvh.plan_chunks(l, c, N, levels)
    descs_dev = kvh.descs_to_tensor(descs, "cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    host_status = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    copy_stream = torch.cuda.Stream()
    want_stream = torch.empty(total, dtype=torch.uint8, device="cuda")
    kvh.encode_chunks(kv, descs_dev, len(descs), want_stream, status, descs=descs)
    n_pages = workloads.n_pages(N)
    table = workloads.shuffled_page_table(n_pages, n_pages + 32, seed=4302).cuda()
    want_pool = kvh.Pool.allocate(l, n_pages + 32, c)
    want_pool.tensor.view(torch.int16).fill_(SENTINEL)
    kvh.decode_batch(want_stream, descs_dev, len(descs), table, want_pool, status)
    assert status.item() == 0

    staging = torch.full((total,), 0x55, dtype=torch.uint8, device="cuda")
    host = torch.full((total,), 0x66, dtype=torch.uint8).pin_memory()
    kvh.store_host(kv, descs, descs_dev, staging, host, status, host_status, copy_stream)
    torch.cuda.current_stream().synchronize()
    assert host_status.item() == 0
    back = torch.empty_like(want_stream)
    back.copy_(host)
    assert torch.equal(back, want_stream), "the stored form in host memory differs from the device encoding"
    del back, kv

    staging.fill_(0x77)
    pool = kvh.Pool.allocate(l, n_pages + 32, c)
    pool.tensor.view(torch.int16).fill_(SENTINEL)
    host_status.fill_(-1)
    kvh.load_host(host, staging, descs, descs_dev, table, pool, status, host_status, copy_stream)
    torch.cuda.synchronize()
    assert host_status.item() == 0
    assert torch.equal(pool.tensor.view(torch.int16), want_pool.tensor.view(torch.int16))
