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
