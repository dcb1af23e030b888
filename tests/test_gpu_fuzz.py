"""Seeded random cases through the whole store/load path on the GPU against the oracle: shapes
(row widths with and without a column-block width, ragged lengths), a level per chunk with and
without the host copy of the descriptors, page sizes, padded pools, shuffled page tables, then a
transcode of every chunk that can go coarser and a decode of the result."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import SENTINEL, kvh, new_status, oracle_pool, sentinel_pool, special_values, from_np16, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu

WIDTHS = [32, 64, 96, 128, 160, 256, 384, 512, 640, 768, 1024, 1152, 1280, 1536, 2048, 2080, 2304]


@pytest.mark.parametrize("seed", range(36))
def test_random_case(kvh, seed):
    rng = np.random.default_rng(1000 + seed)
    c = int(rng.choice(WIDTHS))
    l = int(rng.integers(1, 4))
    N = int(rng.integers(1, 900 if c <= 512 else 400))
    page_tokens = int(rng.choice([16, 16, 32, 64, 8]))
    n_chunks = workloads.n_chunks(N)
    levels = rng.integers(0, 4, size=n_chunks).tolist()
    kv = workloads.make_kv(l, N, c, seed=seed, device="cuda")
    kv_np = to_np16(kv).copy()
    if seed % 3 == 0:
        special_values(kv_np, N)
    kv = from_np16(kv_np)

    want, offsets = oracle.encode_context(kv_np, levels)
    descs, total = kvh.plan_chunks(l, c, N, levels, page_tokens=page_tokens)
    assert total == want.size
    dd = kvh.descs_to_tensor(descs, "cuda")
    status = new_status()
    out = torch.full((total + 128,), 0xA5, dtype=torch.uint8, device="cuda")
    kvh.encode_chunks(kv, dd, n_chunks, out[:total], status, descs=descs if seed % 2 else None)
    g = out.cpu().numpy()
    assert status.item() == 0
    assert np.array_equal(g[:total], want) and np.all(g[total:] == 0xA5)

    npg = -(-N // page_tokens)
    per_chunk = 256 // page_tokens
    num_pages = n_chunks * per_chunk + 3
    perm = workloads.shuffled_page_table(n_chunks * per_chunk, num_pages, seed=seed)
    pad = (int(rng.choice([0, 64])), int(rng.choice([0, 32])), int(rng.choice([0, 8, 40])))
    flat, view, strides = sentinel_pool(l, num_pages, c, page_tokens=page_tokens, pad=pad)
    kvh.decode_batch(out[:total], dd, n_chunks, perm.cuda(), kvh.Pool(view), status)
    ntoks, lv, _ = oracle.chunk_plan(N, levels, l, c)
    want_pool, skipped = oracle_pool(flat.numel(), strides, want, offsets, ntoks, lv, l, c, perm.numpy(), num_pages,
                                     page_tokens)
    assert skipped == 0 and status.item() == 0
    assert np.array_equal(to_np16(flat), want_pool)
    assert npg <= n_chunks * per_chunk

    # every chunk that is not at the coarsest level goes one or more levels down
    go = [i for i, k in enumerate(levels) if k < 3]
    if go and c != 2080:                                 # no column-block width: transcode does not take it
        new_levels = [int(rng.integers(levels[i] + 1, 4)) for i in go]
        din = descs[go].copy()
        dout, total2 = kvh.plan_chunks(l, c, 256 * len(go), new_levels)
        dout["n_tok"] = din["n_tok"]
        want2 = [oracle.transcode_chunk(np.ascontiguousarray(want[offsets[i]:offsets[i + 1]]), levels[i], k, l, c, ntoks[i])
                 for i, k in zip(go, new_levels)]
        out2 = torch.full((total2,), 0x5A, dtype=torch.uint8, device="cuda")
        kvh.transcode(out[:total], kvh.descs_to_tensor(din, "cuda"), out2, kvh.descs_to_tensor(dout, "cuda"), len(go), l, c,
                      -1, -1, status, in_descs=din if seed % 2 else None, out_descs=dout if seed % 2 else None)
        assert status.item() == 0
        o2 = out2.cpu().numpy()
        for j, w in enumerate(want2):
            a = int(dout["stream_off"][j])
            assert np.array_equal(o2[a:a + w.size], w), f"transcoded chunk {go[j]}: {levels[go[j]]} -> {new_levels[j]}"


def test_more_chunks_of_a_level_than_one_list_holds(kvh):
    """A long context of narrow rows: more than 4,000 chunks per level, so the per-level launches
    over chunk lists come in several batches.  Against the oracle on sampled chunks, and against the
    general kernel (no host descriptors) byte for byte."""
    l, c, n_chunks = 1, 32, 8300
    N = 256 * n_chunks - 77
    kv = workloads.make_kv(l, N, c, seed=77, device="cuda")
    levels = [1 if i % 2 else 3 for i in range(n_chunks)]
    descs, total = kvh.plan_chunks(l, c, N, levels)
    dd = kvh.descs_to_tensor(descs, "cuda")
    status = new_status()
    a = torch.full((total,), 0x11, dtype=torch.uint8, device="cuda")
    b = torch.full((total,), 0x22, dtype=torch.uint8, device="cuda")
    kvh.encode_chunks(kv, dd, n_chunks, a, status, descs=descs)
    kvh.encode_chunks(kv, dd, n_chunks, b, status)
    assert status.item() == 0
    assert torch.equal(a, b)
    for i in (0, 3999, 4000, 4001, 8001, n_chunks - 1):
        n = int(descs["n_tok"][i])
        w = oracle.encode_chunk(to_np16(kv[:, :, 256 * i:256 * i + n]), 0, n, levels[i])
        off = int(descs["stream_off"][i])
        assert np.array_equal(a[off:off + w.size].cpu().numpy(), w)
