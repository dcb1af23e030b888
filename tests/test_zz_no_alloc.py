"""The load entry point that allocates nothing (kvh_load_host_static).

Some users of this library cannot allocate device memory at the moment a cache hit has to be
served: a connector living inside a serving engine whose KV pool already owns all free HBM, or a
thread that must stay off the allocator while another part of the process records a CUDA graph.
For them the library stages the stored chunks in a fixed array of its own.  This file checks, through
the C ABI, that such a load fills the pool with exactly the pages the CPU oracle decodes and that
kvh_load_host produces, on two calls in a row (the array is shared and keeps the previous call's
bytes, so the second call would expose stale data if the entry point relied on its contents); that
the device's free memory is the same before and after a call; and that a request larger than the
array, a single chunk of the 70B shape at level 0 included, is refused before anything is enqueued.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import SENTINEL, kvh, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu


def _stored_context(kvh, l, c, N, levels, seed):
    """Encode a seeded context on the GPU and park its stored form in pinned host memory."""
    kv = workloads.make_kv(l, N, c, seed=seed, device="cuda")
    descs, total = kvh.plan_chunks(l, c, N, levels)
    descs_dev = kvh.descs_to_tensor(descs, "cuda")
    streams = torch.empty(total, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kvh.encode_chunks(kv, descs_dev, len(descs), streams, status)
    assert status.item() == 0
    host = torch.empty(total, dtype=torch.uint8).pin_memory()
    host.copy_(streams)
    torch.cuda.synchronize()
    return descs, descs_dev, host, total


def _pool(kvh, l, num_pages, c):
    pool = kvh.Pool.allocate(l, num_pages, c)
    pool.tensor.view(torch.int16).fill_(SENTINEL)
    return pool


def test_static_load_matches_load_host_twice_in_a_row(kvh):
    l, c = 3, 1024
    copy_stream = torch.cuda.Stream()
    dev_status = torch.zeros(1, dtype=torch.int32, device="cuda")
    host_status = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    # two different contexts: lengths, level mixes and page tables differ, so the second call finds
    # the first one's chunks in the shared array at the offsets it is about to use
    cases = [(1500, workloads.chunk_levels(workloads.n_chunks(1500), 4, seed=71), 70, 300_000),
             (1111, [3, 0, 2, 1, 1], 72, 0)]
    first_call = True
    for N, levels, seed, slice_bytes in cases:
        descs, descs_dev, host, total = _stored_context(kvh, l, c, N, levels, seed)
        assert total <= kvh.STATIC_STAGING_BYTES
        npg = workloads.n_pages(N)
        table = workloads.shuffled_page_table(npg, npg + 5, seed=seed).cuda()

        want = _pool(kvh, l, npg + 5, c)
        staging = torch.empty(total, dtype=torch.uint8, device="cuda")
        host_status.fill_(-1)
        kvh.load_host(host, staging, descs, descs_dev, table, want, dev_status, host_status, copy_stream, slice_bytes)
        torch.cuda.synchronize()
        assert host_status.item() == 0

        got = _pool(kvh, l, npg + 5, c)
        host_status.fill_(-1)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        kvh.load_host_static(host, descs, descs_dev, table, got, dev_status, host_status, copy_stream, slice_bytes)
        torch.cuda.synchronize()
        if not first_call:                   # the very first call may load the kernel's code
            assert torch.cuda.mem_get_info()[0] == free_before      # the call took no device memory
        first_call = False
        assert host_status.item() == 0
        a, b = to_np16(got.tensor), to_np16(want.tensor)
        assert np.any(b != SENTINEL)
        assert np.array_equal(a, b)          # decoded pages bit-identical (the tolerance of every parity test here)

        # and both equal what the oracle decodes from the same stored bytes
        ntoks, lv, offsets = oracle.chunk_plan(N, levels, l, c)
        ref = np.full(got.tensor.numel(), SENTINEL, dtype=np.uint16)
        st = got.tensor.stride()
        oracle.decode_context(host.numpy(), offsets, ntoks, lv, l, c, table.cpu().numpy(), ref, st[0], st[1], st[2],
                              npg + 5)
        assert np.array_equal(a.ravel(), ref)


def test_static_load_refuses_what_does_not_fit(kvh):
    l, c, N = 2, 1024, 256
    descs, descs_dev, host, total = _stored_context(kvh, l, c, N, 1, seed=73)
    table = workloads.shuffled_page_table(16, 16, seed=73).cuda()
    pool = _pool(kvh, l, 16, c)
    far = descs.copy()
    far["stream_off"] += kvh.STATIC_STAGING_BYTES - total + 128     # the chunk would end 128 bytes past the array
    copy_stream = torch.cuda.Stream()
    # called through ctypes directly: the Python wrapper would already object to the short host buffer
    st = kvh.lib().kvh_load_host_static(host.data_ptr(), far.ctypes.data, descs_dev.data_ptr(), len(far),
                                        table.data_ptr(), table.numel(), ctypes.byref(pool.struct), None, None,
                                        0, copy_stream.cuda_stream, torch.cuda.current_stream().cuda_stream)
    assert st == 5 and "too small" in kvh.status_string(st)
    # one level-0 chunk of the 70B shape (80 layers x 1024 channels: 80 MiB) is larger than the array,
    # so no split into several calls can serve it; levels 1..3 of the same chunk would fit
    big = kvh.Pool(torch.empty((80, 2, 16, 16, 1024), dtype=torch.bfloat16, device="cuda"))
    one, size = kvh.plan_chunks(80, 1024, 256, 0)
    assert size == 80 << 20 > kvh.STATIC_STAGING_BYTES
    assert all(kvh.plan_chunks(80, 1024, 256, k)[1] <= kvh.STATIC_STAGING_BYTES for k in (1, 2, 3))
    st = kvh.lib().kvh_load_host_static(host.data_ptr(), one.ctypes.data, descs_dev.data_ptr(), 1,
                                        table.data_ptr(), table.numel(), ctypes.byref(big.struct), None, None,
                                        0, copy_stream.cuda_stream, torch.cuda.current_stream().cuda_stream)
    assert st == 5
    torch.cuda.synchronize()
    assert np.all(to_np16(pool.tensor) == SENTINEL)                  # nothing was enqueued
