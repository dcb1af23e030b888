"""Host-tier entry points (stored form in pinned host memory): the bytes that reach the host on
a store and the pages that a load fills must equal the oracle's, whatever the slicing."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import SENTINEL, kvh, oracle_pool, sentinel_pool, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("slice_bytes", [0, 1, 300_000, 1 << 30])
def test_store_then_load_through_pinned_host_memory(kvh, slice_bytes):
    l, c, N = 2, 256, 1500
    kv = workloads.make_kv(l, N, c, seed=31, device="cuda")
    levels = workloads.chunk_levels(workloads.n_chunks(N), 4, seed=32)
    descs, total = kvh.plan_chunks(l, c, N, levels)
    want, offsets = oracle.encode_context(to_np16(kv), levels)
    descs_dev = kvh.descs_to_tensor(descs, "cuda")
    staging = torch.full((total,), 0x55, dtype=torch.uint8, device="cuda")
    host = torch.full((total,), 0x66, dtype=torch.uint8).pin_memory()
    dev_status = torch.zeros(1, dtype=torch.int32, device="cuda")
    host_status = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    copy_stream = torch.cuda.Stream()

    kvh.store_host(kv, descs, descs_dev, staging, host, dev_status, host_status, copy_stream, slice_bytes)
    torch.cuda.current_stream().synchronize()          # the call chains the last copy into this stream
    assert host_status.item() == 0
    assert np.array_equal(host.numpy(), want)

    staging.fill_(0x77)                                # the load must bring every byte back itself
    npg = workloads.n_pages(N)
    table = workloads.shuffled_page_table(npg, npg + 3, seed=33)
    flat, view, strides = sentinel_pool(l, npg + 3, c, pad=(64, 0, 32))
    host_status.fill_(-1)
    kvh.load_host(host, staging, descs, descs_dev, table.cuda(), kvh.Pool(view), dev_status, host_status,
                  copy_stream, slice_bytes)
    torch.cuda.synchronize()
    assert host_status.item() == 0
    ntoks, lv, _ = oracle.chunk_plan(N, levels, l, c)
    want_pool, _ = oracle_pool(flat.numel(), strides, want, offsets, ntoks, lv, l, c, table.numpy(), npg + 3)
    assert np.array_equal(to_np16(flat), want_pool)


def test_host_tier_rejects_gapped_descriptors_and_shared_streams(kvh):
    l, c, N = 1, 64, 600
    kv = workloads.make_kv(l, N, c, seed=34, device="cuda")
    descs, total = kvh.plan_chunks(l, c, N, 2)
    descs_dev = kvh.descs_to_tensor(descs, "cuda")
    staging = torch.empty(total + 4096, dtype=torch.uint8, device="cuda")
    host = torch.empty(total + 4096, dtype=torch.uint8).pin_memory()
    cs = torch.cuda.Stream()
    gapped = descs.copy()
    gapped["stream_off"][2] += 128
    with pytest.raises(kvh.KvhError) as e:
        kvh.store_host(kv, gapped, descs_dev, staging, host, None, None, cs)
    assert e.value.status == 1
    with pytest.raises(kvh.KvhError) as e:
        kvh.store_host(kv, descs, descs_dev, staging[:total - 128], host, None, None, cs)
    assert e.value.status == 5
    with pytest.raises(kvh.KvhError) as e:
        kvh.store_host(kv, descs, descs_dev, staging, host, None, None, torch.cuda.current_stream())
    assert e.value.status == 1
