"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Streams (metadata, codes, padding) must be bit-identical; decoded pages must
be bit-identical too (0 ULP) and every pool element the chunk does not own must keep its
sentinel."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

SENTINEL = 0x7FC1          # a NaN pattern no decode produces from finite inputs


@pytest.fixture(scope="module")
def kvh():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2509_00105_b200 import _build
    _build.build_all()
    import paper_2509_00105_b200 as k
    k.lib()
    return k


def to_np16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_np16(a: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)


def new_status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def sentinel_pool(l, num_pages, c, page_tokens=16, pad=(0, 0, 0)):
    """bf16 pool [l][2][num_pages][page_tokens][c] carved out of a larger sentinel-filled
    buffer so that layers, planes and pages have slack between them."""
    page_stride = page_tokens * c + pad[2]
    kv_stride = num_pages * page_stride + pad[1]
    layer_stride = 2 * kv_stride + pad[0]
    flat = torch.full((l * layer_stride + 64,), SENTINEL, dtype=torch.int16, device="cuda").view(torch.bfloat16)
    view = flat.as_strided((l, 2, num_pages, page_tokens, c), (layer_stride, kv_stride, page_stride, c, 1))
    return flat, view, (layer_stride, kv_stride, page_stride)


def oracle_pool(shape_flat, strides, stream, offsets, ntoks, levels, l, c, page_table, num_pages, page_tokens=16):
    pool = np.full(shape_flat, SENTINEL, dtype=np.uint16)
    skipped = oracle.decode_context(stream, offsets, ntoks, levels, l, c, np.asarray(page_table, dtype=np.int32),
                                    pool, strides[0], strides[1], strides[2], num_pages, page_tokens)
    return pool, skipped


def special_values(kv_np: np.ndarray, seed: int) -> None:
    """Plant signed zeros, subnormals, flat groups, sub-threshold and overflowing ranges."""
    rng = np.random.default_rng(seed)
    l, _, N, c = kv_np.shape
    kv_np[0, 0, 0, 0] = 0x8000
    kv_np[0, 0, min(1, N - 1), 1] = 0x0000
    kv_np[0, 1, 0, :4] = [0x8000, 0x0000, 0x0001, 0x8001]
    if N >= 3:
        kv_np[0, 0, :, 2] = 0x3F80                       # flat K channel
        kv_np[0, 1, 2, :32] = 0xC000                     # flat V group
        kv_np[0, 0, :, 3] = rng.integers(0, 0x80, size=N)            # subnormal K channel: range < 2^-100
        kv_np[0, 1, 1, :32] = rng.choice(np.array([0x7F00, 0xFF00], dtype=np.uint16), size=32)  # +-1.7e38: range overflows
        kv_np[0, 0, :, 4] = rng.choice(np.array([0x0D80, 0x0E00, 0x0E80], dtype=np.uint16), size=N)  # range near 2^-100
        # groups made of signed zeros only: the minimum must be -0 and the maximum +0 when both occur
        kv_np[0, 0, :, 5] = rng.choice(np.array([0x0000, 0x8000], dtype=np.uint16), size=N)
        kv_np[0, 0, :, 6] = np.where(np.arange(N) % 2 == 0, 0x8000, 0x0000)
        kv_np[0, 0, :, 7] = np.where(np.arange(N) % 2 == 0, 0x0000, 0x8000)
        if N >= 6:
            kv_np[0, 1, 5, :32] = rng.choice(np.array([0x0000, 0x8000], dtype=np.uint16), size=32)
        if N >= 5:
            kv_np[0, 1, 3, :32] = np.where(np.arange(32) % 2 == 0, 0x8000, 0x0000)
            kv_np[0, 1, 4, :32] = np.where(np.arange(32) % 2 == 0, 0x0000, 0x8000)


SHAPES = [
    # l, c, N
    (1, 32, 1), (1, 32, 15), (2, 32, 16), (1, 64, 17), (1, 96, 31), (1, 128, 32), (2, 160, 33),
    (1, 256, 255), (1, 32, 256), (2, 64, 257), (1, 1024, 300), (1, 2048, 40), (1, 4096, 33), (3, 512, 700),
    (1, 1152, 70), (1, 1280, 33), (2, 3072, 290), (1, 2080, 35),     # wider than 1024: column blocks of 384, 640, 1024; none
    # rows of at most 512 channels: a work unit takes 2, 4 or 8 tiles; lengths that end a unit after a
    # whole tile, inside its second tile, and that leave whole units empty
    (2, 512, 320), (1, 512, 256 + 33), (1, 384, 200), (1, 256, 2 * 256 + 96), (1, 256, 129), (1, 128, 130),
    (2, 96, 300), (1, 544, 100), (1, 64, 256 + 224),
    # multiples of 256 that are neither: column blocks of 256 channels, four tiles per unit (2-D boxes in the encoder)
    (2, 768, 290), (1, 1280, 256 + 130), (1, 1536, 300), (1, 2304, 97), (1, 1792, 70),
]


@pytest.mark.parametrize("path", ["default", "direct"])
@pytest.mark.parametrize("l,c,N", SHAPES)
@pytest.mark.parametrize("level", [0, 1, 2, 3])
def test_encode_and_decode_match_oracle(kvh, l, c, N, level, path):
    # "default" is the library proper: the persistent TMA-fed encode and decode kernels where they
    # apply; "direct" is the build of the same sources that takes the one-CTA-per-tile kernels on
    # every shape
    kvh = kvh.variant(path)
    assert kvh.build_variant() == path
    kv = workloads.make_kv(l, N, c, seed=1000 * level + N + c, device="cuda")
    kv_np = to_np16(kv).copy()
    special_values(kv_np, N)
    kv = from_np16(kv_np)

    want, offsets = oracle.encode_context(kv_np, level)
    status = new_status()
    out = torch.full((want.size + 256,), 0xAB, dtype=torch.uint8, device="cuda")
    got, total = kvh.encode(kv, level, out=out[:want.size], dev_status=status)
    assert total == want.size
    g = out.cpu().numpy()
    assert np.array_equal(g[:want.size], want)
    assert np.all(g[want.size:] == 0xAB)                 # nothing written past the stream
    assert status.item() == 0

    ntoks, levels, _ = oracle.chunk_plan(N, level, l, c)
    n_pages = workloads.n_pages(N)
    num_pages = n_pages + 5
    table = workloads.shuffled_page_table(n_pages, num_pages, seed=N)
    flat, view, strides = sentinel_pool(l, num_pages, c, pad=(128, 64, 32))
    pool = kvh.Pool(view)
    want_pool, skipped = oracle_pool(flat.numel(), strides, want, offsets, ntoks, levels, l, c, table.numpy(), num_pages)
    assert skipped == 0
    # chunk by chunk through kvh_decode_to_pages ...
    table_dev = table.cuda()
    for i, n in enumerate(ntoks):
        kvh.decode_to_pages(got[offsets[i]:], level, n, table_dev[16 * i:], pool, status)
    assert np.array_equal(to_np16(flat), want_pool)
    # ... and all chunks at once through kvh_decode_batch
    flat.view(torch.int16).fill_(SENTINEL)
    descs, total2 = kvh.plan_chunks(l, c, N, level)
    assert total2 == want.size
    kvh.decode_batch(got, kvh.descs_to_tensor(descs, "cuda"), len(ntoks), table_dev, pool, status)
    assert np.array_equal(to_np16(flat), want_pool)
    assert status.item() == 0


def test_tiny_config_every_level(kvh):
    """The small benchmark configuration: l=4, N=256, c=1024, seed 0, full oracle parity."""
    s = workloads.TINY
    kv = workloads.make_kv(s.n_layers, s.n_tokens, s.n_channels, seed=0, device="cuda")
    kv_np = to_np16(kv)
    table = workloads.shuffled_page_table(16, 64, seed=0)
    for level in range(4):
        want, offsets = oracle.encode_context(kv_np, level)
        got, total = kvh.encode(kv, level)
        assert np.array_equal(got.cpu().numpy(), want)
        flat, view, strides = sentinel_pool(s.n_layers, 64, s.n_channels)
        kvh.decode_to_pages(got, level, 256, table.cuda(), kvh.Pool(view))
        want_pool, _ = oracle_pool(flat.numel(), strides, want, offsets, [256], [level], s.n_layers, s.n_channels,
                                   table.numpy(), 64)
        assert np.array_equal(to_np16(flat), want_pool)
        if level == 0:                                   # lossless: pages hold the input bits
            p = to_np16(view)
            for pg in range(16):
                assert np.array_equal(p[:, :, table[pg]], kv_np[:, :, 16 * pg:16 * pg + 16])


def test_batched_mixed_level_decode_into_shared_pool(kvh):
    """Several contexts with ragged lengths, a random level per chunk, one shuffled page table,
    one launch (the structure of the batched-load workload, scaled down)."""
    l, c = 2, 256
    lengths = [300, 256, 1, 777, 40, 512, 129]
    num_pages = sum(workloads.n_pages(n) for n in lengths) + 9
    perm = workloads.shuffled_page_table(num_pages - 9, num_pages, seed=5)
    flat, view, strides = sentinel_pool(l, num_pages, c, pad=(0, 0, 0))
    want_pool = np.full(flat.numel(), SENTINEL, dtype=np.uint16)
    streams, all_descs, tables = [], [], []
    stream_base = pt_base = 0
    status = new_status()
    for i, N in enumerate(lengths):
        kv = workloads.make_kv(l, N, c, seed=50 + i, device="cuda")
        kv_np = to_np16(kv)
        levels = workloads.chunk_levels(workloads.n_chunks(N), 4, seed=70 + i)
        want, offsets = oracle.encode_context(kv_np, levels)
        descs, total = kvh.plan_chunks(l, c, N, levels, stream_base=stream_base, pt_base=pt_base)
        assert total == want.size
        # mixed-level encode through kvh_encode_chunks, into a buffer local to the context
        local, _ = kvh.plan_chunks(l, c, N, levels)
        out = torch.full((total,), 0xCD, dtype=torch.uint8, device="cuda")
        kvh.encode_chunks(kv, kvh.descs_to_tensor(local, "cuda"), len(levels), out, status)
        assert np.array_equal(out.cpu().numpy(), want)
        # the same with the host copy of the descriptors: one specialised launch per level
        out.fill_(0xCD)
        kvh.encode_chunks(kv, kvh.descs_to_tensor(local, "cuda"), len(levels), out, status, descs=local)
        assert np.array_equal(out.cpu().numpy(), want)
        npg = workloads.n_pages(N)
        ids = perm[pt_base:pt_base + npg]
        ntoks, lv, _ = oracle.chunk_plan(N, levels, l, c)
        oracle.decode_context(want, offsets, ntoks, lv, l, c, ids.numpy(), want_pool, *strides, num_pages)
        streams.append(out)
        all_descs.append(descs)
        stream_base += total
        pt_base += npg
    descs = np.concatenate(all_descs)
    blob = torch.cat(streams)
    kvh.decode_batch(blob, kvh.descs_to_tensor(descs, "cuda"), len(descs), perm.cuda(), kvh.Pool(view), status)
    assert status.item() == 0
    assert np.array_equal(to_np16(flat), want_pool)


def test_out_of_range_page_is_skipped_and_reported(kvh):
    l, c, N = 2, 64, 100
    kv = workloads.make_kv(l, N, c, seed=8, device="cuda")
    got, _ = kvh.encode(kv, 2)
    want, offsets = oracle.encode_context(to_np16(kv), 2)
    num_pages = 10
    ids = np.array([3, 10, 0, -1, 9, 2, 1], dtype=np.int32)      # entries 1 and 3 are outside [0, 10)
    flat, view, strides = sentinel_pool(l, num_pages, c, pad=(64, 64, 64))
    status = new_status()
    kvh.decode_to_pages(got, 2, N, torch.from_numpy(ids).cuda(), kvh.Pool(view), status)
    want_pool, skipped = oracle_pool(flat.numel(), strides, want, offsets, [N], [2], l, c, ids, num_pages)
    assert skipped == 32 * l * 2
    assert status.item() == 6
    assert np.array_equal(to_np16(flat), want_pool)


@pytest.mark.parametrize("level", [0, 1, 2, 3])
def test_out_of_range_pages_in_whole_tiles_at_the_compiled_in_width(kvh, level):
    """Rows of 1024 channels and whole tiles take the unrolled consumers whose warps step through a
    tile's rows behind a named barrier.  A page id outside the pool must make exactly the threads
    that own its rows skip their stores: every other page is written, nothing else is touched, the
    status says so, and every thread still reaches every barrier (the launch ends)."""
    l, c, N = 2, 1024, 512
    kv = workloads.make_kv(l, N, c, seed=80 + level, device="cuda")
    got, _ = kvh.encode(kv, level)
    want, offsets = oracle.encode_context(to_np16(kv), level)
    assert np.array_equal(got.cpu().numpy(), want)
    num_pages = 40
    ids = workloads.shuffled_page_table(32, num_pages, seed=81).numpy().copy()
    ids[[0, 5, 17, 31]] = [num_pages, -1, 1 << 30, num_pages + 7]      # first page of a tile, second page, both chunks
    descs, _ = kvh.plan_chunks(l, c, N, level)
    flat, view, strides = sentinel_pool(l, num_pages, c, pad=(128, 64, 32))
    status = new_status()
    kvh.decode_batch(got, kvh.descs_to_tensor(descs, "cuda"), len(descs), torch.from_numpy(ids).cuda(), kvh.Pool(view), status)
    torch.cuda.synchronize()
    want_pool, skipped = oracle_pool(flat.numel(), strides, want, offsets, [256, 256], [level, level], l, c, ids, num_pages)
    assert skipped == 4 * 16 * l * 2
    assert status.item() == 6
    assert np.array_equal(to_np16(flat), want_pool)


def test_bad_descriptors_are_skipped_and_reported(kvh):
    l, c, N = 1, 64, 512
    kv = workloads.make_kv(l, N, c, seed=9, device="cuda")
    descs, total = kvh.plan_chunks(l, c, N, [1, 3])
    out = torch.zeros(total, dtype=torch.uint8, device="cuda")
    kvh.encode_chunks(kv, kvh.descs_to_tensor(descs, "cuda"), 2, out)
    want, offsets = oracle.encode_context(to_np16(kv), [1, 3])
    assert np.array_equal(out.cpu().numpy(), want)
    table = torch.arange(32, dtype=torch.int32, device="cuda")

    def run(mutate, expect):
        d = descs.copy()
        mutate(d)
        flat, view, strides = sentinel_pool(l, 32, c)
        status = new_status()
        kvh.decode_batch(out, kvh.descs_to_tensor(d, "cuda"), 2, table, kvh.Pool(view), status)
        assert status.item() == expect
        # chunk 0 stays good in every case: its pages match the oracle, chunk 1's stay untouched
        wp, _ = oracle_pool(flat.numel(), strides, want, offsets, [256], [1], l, c, np.arange(32), 32)
        assert np.array_equal(to_np16(flat), wp)

    run(lambda d: d["level"].__setitem__(1, 9), 2)
    run(lambda d: d["n_tok"].__setitem__(1, 0), 3)
    run(lambda d: d["stream_off"].__setitem__(1, d["stream_off"][1] + 8), 4)
    run(lambda d: d["stream_off"].__setitem__(1, total), 5)
    run(lambda d: d["pt_off"].__setitem__(1, 30), 5)
    run(lambda d: d["pt_off"].__setitem__(1, -4), 5)

    # encode side: a descriptor whose token count disagrees with the context is skipped
    d = descs.copy()
    d["n_tok"][1] = 100
    status = new_status()
    out2 = torch.full((total,), 0xEE, dtype=torch.uint8, device="cuda")
    kvh.encode_chunks(kv, kvh.descs_to_tensor(d, "cuda"), 2, out2, status)
    assert status.item() == 3
    o = out2.cpu().numpy()
    assert np.array_equal(o[:offsets[1]], want[:offsets[1]]) and np.all(o[offsets[1]:] == 0xEE)
    # and one that would run past the output buffer
    status = new_status()
    out3 = torch.full((total,), 0xEE, dtype=torch.uint8, device="cuda")
    kvh.encode_chunks(kv, kvh.descs_to_tensor(descs, "cuda"), 2, out3[:total - 128], status)
    assert status.item() == 5
    assert np.all(out3.cpu().numpy()[offsets[1]:] == 0xEE)


@pytest.mark.parametrize("path", ["default", "direct"])
@pytest.mark.parametrize("l,c,N", [(1, 64, 100), (2, 1024, 300), (1, 2048, 77), (2, 512, 600), (1, 128, 333)])
def test_page_size_other_than_16(kvh, l, c, N, path):
    """Pages of 8 tokens and more go through the persistent kernel (a thread's run of rows is cut at
    page boundaries: a 32-token tile then spans up to 4 pages); smaller pages take the direct one."""
    kvh = kvh.variant(path)
    kv = workloads.make_kv(l, N, c, seed=12, device="cuda")
    for page_tokens in (4, 8, 32, 64, 256):
        for level in (0, 1, 3):
            got, _ = kvh.encode(kv, level)
            want, offsets = oracle.encode_context(to_np16(kv), level)
            per_chunk = 256 // page_tokens
            n_chunks = workloads.n_chunks(N)
            ids = torch.randperm(n_chunks * per_chunk + 2, generator=torch.Generator().manual_seed(3))[:n_chunks * per_chunk].to(torch.int32)
            flat, view, strides = sentinel_pool(l, n_chunks * per_chunk + 2, c, page_tokens=page_tokens)
            descs, _ = kvh.plan_chunks(l, c, N, level, page_tokens=page_tokens)
            status = new_status()
            kvh.decode_batch(got, kvh.descs_to_tensor(descs, "cuda"), n_chunks, ids.cuda(), kvh.Pool(view), status)
            ntoks, lv, _ = oracle.chunk_plan(N, level, l, c)
            wp, _ = oracle_pool(flat.numel(), strides, want, offsets, ntoks, lv, l, c, ids.numpy(), n_chunks * per_chunk + 2,
                                page_tokens)
            assert status.item() == 0
            assert np.array_equal(to_np16(flat), wp), f"page_tokens {page_tokens} level {level}"


def test_gpu_decodes_oracle_streams_and_oracle_decodes_gpu_streams(kvh):
    """Cross-decoding: each side's stream is a valid input of the other (they are identical, so
    this mostly guards the comparison helpers themselves)."""
    l, c, N = 2, 128, 200
    kv = workloads.make_kv(l, N, c, seed=21, device="cuda")
    for level in (1, 2, 3):
        want, offsets = oracle.encode_context(to_np16(kv), level)
        flat, view, strides = sentinel_pool(l, 16, c)
        ids = torch.arange(15, -1, -1, dtype=torch.int32)
        kvh.decode_to_pages(torch.from_numpy(want).cuda(), level, N, ids.cuda(), kvh.Pool(view))
        got, _ = kvh.encode(kv, level)
        wp, _ = oracle_pool(flat.numel(), strides, got.cpu().numpy(), offsets, [N], [level], l, c, ids.numpy(), 16)
        assert np.array_equal(to_np16(flat), wp)


def lattice_kv(l, N, c, seed):
    """Values on small integer lattices times a power of two: within a group x - min and max - min
    are small integers, so (x - min) * qmax / (max - min) lands exactly on k + 1/2 very often while
    qmax / (max - min) is inexact.  Any evaluation that does not round the product before rounding to
    an integer (a fused multiply-add) then picks the wrong neighbour."""
    rng = np.random.default_rng(seed)
    span = rng.integers(1, 256, size=(l, 2, (N + 31) // 32, 1, c // 32, 1))          # per 32 x 32 block
    m = rng.integers(0, 256, size=(l, 2, (N + 31) // 32, 32, c // 32, 32)) % (span + 1)
    m[:, :, :, 0, :, 0] = 0                                   # every K column and V row of a block sees 0 ...
    m[:, :, :, :, :, 1] = np.where(np.arange(32)[None, None, None, :, None] % 2 == 0, 0, span[..., 0])
    m[:, :, :, 1, :, :] = np.where(np.arange(32) % 2 == 0, span[:, :, :, 0, :, :], 0)   # ... and the block's span
    e = rng.integers(-6, 7, size=(l, 2, (N + 31) // 32, 1, c // 32, 1))
    x = (m * (2.0 ** e)).astype(np.float32).reshape(l, 2, -1, c // 32, 32)
    x = x.reshape(l, 2, -1, c)[:, :, :N]
    bits = np.ascontiguousarray(x).view(np.uint32)
    assert np.all((bits & 0xFFFF) == 0)                       # exact in bf16
    return (bits >> 16).astype(np.uint16)


@pytest.mark.parametrize("l,c,N", [(2, 1024, 512), (1, 64, 300), (1, 2048, 64), (1, 256, 300)])
@pytest.mark.parametrize("level", [1, 2, 3])
def test_encode_rounds_ties_like_the_oracle(kvh, l, c, N, level):
    kv_np = lattice_kv(l, N, c, seed=level * 100 + c)
    want, _ = oracle.encode_context(kv_np, level)
    got, _ = kvh.encode(from_np16(kv_np), level)
    assert np.array_equal(got.cpu().numpy(), want)


def test_mixed_level_encode_with_host_descriptors(kvh):
    """c = 1024, many chunks, every level: per-level launches over chunk lists must produce the same
    stream as the oracle; a chunk whose host and device descriptors disagree is skipped and reported."""
    l, c, N = 2, 1024, 256 * 37 + 100
    kv = workloads.make_kv(l, N, c, seed=91, device="cuda")
    levels = workloads.chunk_levels(workloads.n_chunks(N), 4, seed=92)
    assert set(levels) == {0, 1, 2, 3}
    want, offsets = oracle.encode_context(to_np16(kv), levels)
    descs, total = kvh.plan_chunks(l, c, N, levels)
    out = torch.full((total,), 0xCD, dtype=torch.uint8, device="cuda")
    status = new_status()
    kvh.encode_chunks(kv, kvh.descs_to_tensor(descs, "cuda"), len(descs), out, status, descs=descs)
    assert status.item() == 0
    assert np.array_equal(out.cpu().numpy(), want)
    # chunk 5: the host says another level than the device; chunk 7: the host names no level at all
    lie = descs.copy()
    lie["level"][5] = (levels[5] + 1) % 4
    lie["level"][7] = 9
    out.fill_(0xCD)
    kvh.encode_chunks(kv, kvh.descs_to_tensor(descs, "cuda"), len(descs), out, status, descs=lie)
    assert status.item() == 2
    o = out.cpu().numpy()
    for i in range(len(descs)):
        a, b = offsets[i], offsets[i + 1]
        if i == 5:
            assert np.all(o[a:b] == 0xCD)
        else:                                            # chunk 7 is encoded by the general kernel from its device descriptor
            assert np.array_equal(o[a:b], want[a:b])
