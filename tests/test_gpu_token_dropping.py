"""Token dropping on the GPU (kvh_encode_kept) against the oracle: the stored streams of the kept
tokens must be bit-identical to the oracle's encoding of the compacted tensor, and decoding them
fills consecutive page slots with the kept tokens."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import SENTINEL, kvh, new_status, oracle_pool, sentinel_pool, special_values, from_np16, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu

CASES = [
    # l, c, N, runs (None = sinks + recent), levels
    (1, 1024, 700, [(0, 4), (444, 256)], 3),             # seam inside the first tile
    (2, 1024, 2000, [(0, 4), (1000, 700)], [1, 3, 0]),   # mixed levels over the kept chunks
    (1, 256, 900, [(0, 1), (100, 31), (131, 1), (500, 300)], 2),     # adjacent runs, odd lengths
    (1, 32, 4000, [(50 * i * i + 3 * i, 37 + i) for i in range(8)], [2, 0]),  # the most runs the call accepts
    (2, 512, 300, [(0, 300)], 1),                        # nothing dropped
    (1, 1024, 5000, [(4999, 1)], 3),                     # a single kept token
    (1, 64, 600, [(0, 33), (567, 33)], 0),               # level 0: kept rows as they are
    (1, 2048, 300, [(0, 4), (100, 60)], 2),              # rows wider than a stage: column blocks of 1024
    (1, 1152, 200, [(3, 30), (150, 41)], [1]),           # ... of 384
    (1, 3072, 90, [(0, 90)], 0),
    (2, 512, 1500, [(0, 4), (700, 350), (1100, 90)], [3, 1]),        # narrow rows: seams inside units of two tiles
    (1, 128, 3000, [(5, 100), (1000, 7), (2000, 333)], 2),           # ... of eight
    (1, 768, 500, [(0, 4), (200, 290)], [1, 3]),                     # a width the plain encoder takes in 2-D boxes: rows gathered instead
    (1, 1280, 300, [(10, 33), (100, 100)], 2),
]


@pytest.mark.parametrize("l,c,N,runs,levels", CASES)
def test_encode_kept_matches_oracle(kvh, l, c, N, runs, levels):
    kv = workloads.make_kv(l, N, c, seed=N + c, device="cuda")
    kv_np = to_np16(kv).copy()
    special_values(kv_np, N)
    kv = from_np16(kv_np)
    n_kept = sum(n for _, n in runs)
    want, offsets = oracle.encode_kept(kv_np, runs, levels)
    descs, total = kvh.plan_chunks(l, c, n_kept, levels)
    assert total == want.size
    out = torch.full((total + 256,), 0xAB, dtype=torch.uint8, device="cuda")
    status = new_status()
    kvh.encode_kept(kv, np.array(runs, dtype=kvh.RUN_DTYPE), kvh.descs_to_tensor(descs, "cuda"), len(descs),
                    out[:total], status)
    g = out.cpu().numpy()
    assert status.item() == 0
    assert np.array_equal(g[:total], want)
    assert np.all(g[total:] == 0xAB)
    if isinstance(levels, int):                          # one level: the specialised kernel, with and without descriptors
        for dd in (kvh.descs_to_tensor(descs, "cuda"), None):
            out.fill_(0xAB)
            kvh.encode_kept(kv, np.array(runs, dtype=kvh.RUN_DTYPE), dd, len(descs), out[:total], status, level=levels)
            g = out.cpu().numpy()
            assert status.item() == 0
            assert np.array_equal(g[:total], want) and np.all(g[total:] == 0xAB)

    # a hit loads the kept tokens into consecutive page slots
    npg = workloads.n_pages(n_kept)
    table = workloads.shuffled_page_table(npg, npg + 3, seed=N)
    flat, view, strides = sentinel_pool(l, npg + 3, c, pad=(64, 0, 32))
    kvh.decode_batch(out[:total], kvh.descs_to_tensor(descs, "cuda"), len(descs), table.cuda(), kvh.Pool(view), status)
    ntoks, lv, _ = oracle.chunk_plan(n_kept, levels, l, c)
    want_pool, _ = oracle_pool(flat.numel(), strides, want, offsets, ntoks, lv, l, c, table.numpy(), npg + 3)
    assert status.item() == 0
    assert np.array_equal(to_np16(flat), want_pool)


def test_sinks_and_recent_window_at_benchmark_shape(kvh):
    """The 8B-shaped context (l=32, c=1024, N=8192) with 4 sink tokens and a 2044-token recent
    window (rate 1/4), 2-bit: sampled chunks against the oracle."""
    s = workloads.LLAMA8B_8K
    l, c, N = s.n_layers, s.n_channels, s.n_tokens
    kv = workloads.make_kv(l, N, c, seed=6000, device="cuda")
    runs, n_kept = kvh.keep_sinks_and_recent(N, 4, 2044)
    assert n_kept == 2048 and [(int(r["first"]), int(r["count"])) for r in runs] == oracle.keep_sinks_and_recent(N, 4, 2044)
    descs, total = kvh.plan_chunks(l, c, n_kept, 3)
    assert total * 4 == kvh.plan_chunks(l, c, N, 3)[1]                   # size = rate x size
    out = torch.empty(total, dtype=torch.uint8, device="cuda")
    status = new_status()
    kvh.encode_kept(kv, runs, None, len(descs), out, status, level=3)
    assert status.item() == 0
    compact = torch.cat([kv[:, :, :4], kv[:, :, N - 2044:]], dim=2)
    for i in (0, 3, 7):                                  # chunk 0 holds the seam
        want = oracle.encode_chunk(to_np16(compact[:, :, 256 * i:256 * i + 256]), 0, 256, 3)
        off = int(descs["stream_off"][i])
        assert np.array_equal(out[off:off + want.size].cpu().numpy(), want)


def test_encode_kept_rejects_bad_runs(kvh):
    l, c, N = 1, 64, 600
    kv = workloads.make_kv(l, N, c, seed=1, device="cuda")
    descs, total = kvh.plan_chunks(l, c, 100, 1)
    dd = kvh.descs_to_tensor(descs, "cuda")
    out = torch.empty(total, dtype=torch.uint8, device="cuda")
    R = lambda runs: np.array(runs, dtype=kvh.RUN_DTYPE)
    for runs, status in (([(0, 50), (40, 50)], 1), ([(0, 0), (5, 100)], 1), ([(550, 100)], 1), ([(0, 300)], 3),
                         ([(i, 1) for i in range(0, 18, 2)], 1)):
        with pytest.raises(kvh.KvhError) as e:
            kvh.encode_kept(kv, R(runs), dd, len(descs), out)
        assert e.value.status == status
    # the chunk count fits but a descriptor's token count does not: the kernel skips it and says so
    status = new_status()
    out.fill_(0xEE)
    kvh.encode_kept(kv, R([(0, 99)]), dd, len(descs), out, status)
    assert status.item() == 3 and bool((out == 0xEE).all())
    # a level is announced and a descriptor has another one
    status = new_status()
    kvh.encode_kept(kv, R([(0, 100)]), dd, len(descs), out, status, level=2)
    assert status.item() == 2
    with pytest.raises(kvh.KvhError) as e:               # neither descriptors nor a level
        kvh.encode_kept(kv, R([(0, 100)]), None, len(descs), out)
    assert e.value.status == 1
    with pytest.raises(kvh.KvhError) as e:
        kvh.encode_kept(kv, R([(0, 100)]), None, len(descs), out[:total - 128], level=1)
    assert e.value.status == 5
    wide = workloads.make_kv(1, 40, 2080, seed=2, device="cuda")      # 65 x 32 channels: no column-block width fits
    d2, t2 = kvh.plan_chunks(1, 2080, 8, 1)
    with pytest.raises(kvh.KvhError) as e:
        kvh.encode_kept(wide, R([(0, 8)]), kvh.descs_to_tensor(d2, "cuda"), 1, torch.empty(t2, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
