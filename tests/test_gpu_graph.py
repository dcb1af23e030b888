"""The store and load calls inside a CUDA graph: they allocate nothing and only enqueue work on
the caller's stream, so a serving engine can capture them once and replay them.  The replay must
produce what the oracle produces for whatever the input buffers hold at replay time."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import SENTINEL, kvh, new_status, oracle_pool, sentinel_pool, from_np16, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu


def test_encode_and_batched_decode_replayed_from_a_graph(kvh):
    l, c, N = 2, 1024, 700
    levels = [3, 1, 2]
    descs, total = kvh.plan_chunks(l, c, N, levels)
    dd = kvh.descs_to_tensor(descs, "cuda")
    npg = workloads.n_pages(N)
    table = workloads.shuffled_page_table(npg, npg + 2, seed=4)
    table_dev = table.cuda()
    flat, view, strides = sentinel_pool(l, npg + 2, c)
    pool = kvh.Pool(view)
    kv = workloads.make_kv(l, N, c, seed=40, device="cuda")
    out = torch.zeros(total, dtype=torch.uint8, device="cuda")
    status = new_status()
    # once eagerly (also sets the kernels' shared-memory attributes), then captured
    kvh.encode_chunks(kv, dd, len(descs), out, status, descs=descs)
    kvh.decode_batch(out, dd, len(descs), table_dev, pool, status)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        kvh.encode_chunks(kv, dd, len(descs), out, status, descs=descs)
        kvh.decode_batch(out, dd, len(descs), table_dev, pool, status)
    for seed in (41, 42):
        kv.copy_(workloads.make_kv(l, N, c, seed=seed, device="cuda"))
        out.zero_()
        flat.view(torch.int16).fill_(SENTINEL)
        graph.replay()
        torch.cuda.synchronize()
        want, offsets = oracle.encode_context(to_np16(kv), levels)
        assert status.item() == 0
        assert np.array_equal(out.cpu().numpy(), want)
        ntoks, lv, _ = oracle.chunk_plan(N, levels, l, c)
        want_pool, _ = oracle_pool(flat.numel(), strides, want, offsets, ntoks, lv, l, c, table.numpy(), npg + 2)
        assert np.array_equal(to_np16(flat), want_pool)


def test_token_dropping_and_transcode_replayed_from_a_graph(kvh):
    """Store with dropped tokens at 8 bits, then compress the stored chunks further to 2 bits, both
    captured once and replayed on new contents (rows of 512 channels: units of two tiles)."""
    l, c, N = 2, 512, 1100
    runs = [(0, 4), (300, 500), (1000, 100)]
    n_kept = sum(n for _, n in runs)
    runs_np = np.array(runs, dtype=kvh.RUN_DTYPE)
    d1, total1 = kvh.plan_chunks(l, c, n_kept, 1)
    d3, total3 = kvh.plan_chunks(l, c, n_kept, 3)
    dd1, dd3 = kvh.descs_to_tensor(d1, "cuda"), kvh.descs_to_tensor(d3, "cuda")
    kv = workloads.make_kv(l, N, c, seed=50, device="cuda")
    s1 = torch.zeros(total1, dtype=torch.uint8, device="cuda")
    s3 = torch.zeros(total3, dtype=torch.uint8, device="cuda")
    status = new_status()

    def step():
        kvh.encode_kept(kv, runs_np, dd1, len(d1), s1, status, level=1)
        kvh.transcode(s1, dd1, s3, dd3, len(d1), l, c, 1, 3, dev_status=status)

    step()                                               # eagerly once (kernel attributes), then captured
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for seed in (51, 52):
        kv.copy_(workloads.make_kv(l, N, c, seed=seed, device="cuda"))
        s1.zero_()
        s3.zero_()
        graph.replay()
        torch.cuda.synchronize()
        want1, offsets = oracle.encode_kept(to_np16(kv), runs, 1)
        ntoks, _, _ = oracle.chunk_plan(n_kept, 1, l, c)
        want3 = np.concatenate([oracle.transcode_chunk(np.ascontiguousarray(want1[offsets[i]:offsets[i + 1]]), 1, 3, l, c, n)
                                for i, n in enumerate(ntoks)])
        assert status.item() == 0
        assert np.array_equal(s1.cpu().numpy(), want1)
        assert np.array_equal(s3.cpu().numpy(), want3)
