"""Transcoding on the GPU (kvh_transcode) against the oracle: the new stream must equal, bit for
bit, the oracle's encoding at the new level of what the old stream decodes to."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import kvh, new_status, special_values, from_np16, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu

PAIRS = [(0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3)]


def oracle_transcode_context(stream, offsets, ntoks, levels_in, levels_out, l, c):
    parts = [oracle.transcode_chunk(np.ascontiguousarray(stream[offsets[i]:offsets[i + 1]]), levels_in[i],
                                    levels_out[i], l, c, n) for i, n in enumerate(ntoks)]
    return np.concatenate(parts)


def run_case(kvh, l, c, N, levels_in, levels_out, hint):
    kv = workloads.make_kv(l, N, c, seed=7 * N + c, device="cuda")
    kv_np = to_np16(kv).copy()
    special_values(kv_np, N)
    src, offsets = oracle.encode_context(kv_np, levels_in)
    ntoks, lin, _ = oracle.chunk_plan(N, levels_in, l, c)
    _, lout, _ = oracle.chunk_plan(N, levels_out, l, c)
    want = oracle_transcode_context(src, offsets, ntoks, lin, lout, l, c)
    din, _ = kvh.plan_chunks(l, c, N, levels_in)
    dout, total = kvh.plan_chunks(l, c, N, levels_out)
    assert total == want.size
    out = torch.full((total + 256,), 0xAB, dtype=torch.uint8, device="cuda")
    status = new_status()
    kvh.transcode(torch.from_numpy(src).cuda(), kvh.descs_to_tensor(din, "cuda"), out[:total],
                  kvh.descs_to_tensor(dout, "cuda"), len(din), l, c, *hint, dev_status=status)
    g = out.cpu().numpy()
    assert status.item() == 0
    assert np.array_equal(g[:total], want)
    assert np.all(g[total:] == 0xAB)
    if hint == (-1, -1):                                 # with the host descriptors: one launch per pair of levels
        out.fill_(0xAB)
        kvh.transcode(torch.from_numpy(src).cuda(), kvh.descs_to_tensor(din, "cuda"), out[:total],
                      kvh.descs_to_tensor(dout, "cuda"), len(din), l, c, -1, -1, dev_status=status,
                      in_descs=din, out_descs=dout)
        g = out.cpu().numpy()
        assert status.item() == 0
        assert np.array_equal(g[:total], want) and np.all(g[total:] == 0xAB)


@pytest.mark.parametrize("l,c,N", [(1, 1024, 300), (2, 256, 257), (1, 32, 33), (1, 96, 700), (2, 1024, 64),
                                   (1, 2048, 70), (1, 1152, 40),
                                   (2, 512, 320), (1, 512, 289), (1, 128, 256 + 130), (1, 384, 200)])   # units of 2, 8 and 2 tiles
@pytest.mark.parametrize("pair", PAIRS)
def test_transcode_one_pair_of_levels(kvh, l, c, N, pair):
    run_case(kvh, l, c, N, pair[0], pair[1], pair)       # the kernel specialised for the pair
    run_case(kvh, l, c, N, pair[0], pair[1], (-1, -1))   # and the one that takes any mix


def test_transcode_mixed_levels(kvh):
    N = 256 * 6 + 45
    run_case(kvh, 2, 1024, N, [0, 0, 0, 1, 1, 2, 1], [1, 2, 3, 2, 3, 3, 3], (-1, -1))
    run_case(kvh, 1, 64, N, [2, 1, 0, 0, 1, 0, 0], [3, 3, 3, 1, 2, 2, 1], (-1, -1))


def test_transcode_skips_and_reports_chunks_that_break_a_rule(kvh):
    l, c, N = 1, 64, 512
    kv = workloads.make_kv(l, N, c, seed=3, device="cuda")
    src, _ = kvh.encode(kv, 1)
    din, _ = kvh.plan_chunks(l, c, N, 1)
    dout, total = kvh.plan_chunks(l, c, N, 3)
    want = oracle_transcode_context(src.cpu().numpy(), [0, int(din["stream_off"][1]), src.numel()], [256, 256],
                                    [1, 1], [3, 3], l, c)
    half = int(dout["stream_off"][1])

    room = kvh.level_bytes(0, l, c, 256)

    def run(mut_in, mut_out, expect, hint=(-1, -1), capacity=None):
        a, b = din.copy(), dout.copy()
        mut_in(a); mut_out(b)
        out = torch.full((total + room,), 0xEE, dtype=torch.uint8, device="cuda")    # room for a chunk at any level
        status = new_status()
        kvh.transcode(src, kvh.descs_to_tensor(a, "cuda"), out[:capacity or total + room], kvh.descs_to_tensor(b, "cuda"),
                      2, l, c, *hint, dev_status=status)
        o = out.cpu().numpy()
        assert status.item() == expect
        assert np.array_equal(o[:half], want[:half]) and np.all(o[half:] == 0xEE)   # chunk 0 fine, chunk 1 untouched
        if hint == (-1, -1):                             # the same when the host knows the descriptors
            out.fill_(0xEE)
            status.zero_()
            kvh.transcode(src, kvh.descs_to_tensor(a, "cuda"), out[:capacity or total + room], kvh.descs_to_tensor(b, "cuda"),
                          2, l, c, -1, -1, dev_status=status, in_descs=a, out_descs=b)
            o = out.cpu().numpy()
            assert status.item() == expect
            assert np.array_equal(o[:half], want[:half]) and np.all(o[half:] == 0xEE)

    nop = lambda d: None
    run(nop, lambda d: d["level"].__setitem__(1, 1), 2)              # not coarser
    run(nop, lambda d: d["level"].__setitem__(1, 0), 2)              # finer
    run(nop, lambda d: d["n_tok"].__setitem__(1, 255), 3)            # token counts disagree
    run(lambda d: d["stream_off"].__setitem__(1, src.numel()), nop, 5)
    run(nop, nop, 5, capacity=total - 128)                           # the new chunk would not fit
    run(nop, lambda d: d["level"].__setitem__(1, 2), 2, hint=(1, 3))  # not the announced pair
    for hint in ((3, 1), (1, 1), (1, -1), (0, 4)):
        with pytest.raises(kvh.KvhError) as e:
            kvh.transcode(src, kvh.descs_to_tensor(din, "cuda"), torch.empty(total, dtype=torch.uint8, device="cuda"),
                          kvh.descs_to_tensor(dout, "cuda"), 2, l, c, *hint)
        assert e.value.status == 2


def test_transcode_at_benchmark_shape(kvh):
    """The 8B-shaped context (l=32, c=1024, N=8192): 8 bit -> 2 bit, sampled chunks against the oracle,
    and equal to what decoding into pages and encoding those pages again gives."""
    s = workloads.LLAMA8B_8K
    l, c, N = s.n_layers, s.n_channels, s.n_tokens
    kv = workloads.make_kv(l, N, c, seed=7000, device="cuda")
    src, _ = kvh.encode(kv, 1)
    din, _ = kvh.plan_chunks(l, c, N, 1)
    dout, total = kvh.plan_chunks(l, c, N, 3)
    out = torch.empty(total, dtype=torch.uint8, device="cuda")
    status = new_status()
    kvh.transcode(src, kvh.descs_to_tensor(din, "cuda"), out, kvh.descs_to_tensor(dout, "cuda"), len(din), l, c, 1, 3,
                  dev_status=status)
    assert status.item() == 0
    for i in (0, 17, 31):
        a, b = int(din["stream_off"][i]), int(dout["stream_off"][i])
        want = oracle.transcode_chunk(src[a:a + kvh.level_bytes(1, l, c, 256)].cpu().numpy(), 1, 3, l, c, 256)
        assert np.array_equal(out[b:b + want.size].cpu().numpy(), want)
    # the long way round on the GPU: decode into an identity-mapped pool, encode the pool's rows
    pool = kvh.Pool.allocate(l, N // 16, c)
    kvh.decode_batch(src, kvh.descs_to_tensor(din, "cuda"), len(din), torch.arange(N // 16, dtype=torch.int32, device="cuda"),
                     pool, status)
    again, _ = kvh.encode(pool.tensor.view(l, 2, N, c), 3)
    assert torch.equal(again, out)


@pytest.mark.parametrize("pair", PAIRS)
def test_transcode_rounds_ties_like_the_oracle(kvh, pair):
    """Sources on integer lattices (see lattice_kv): re-quantising hits exact ties all the time."""
    from test_gpu_parity import lattice_kv
    l, c, N = 2, 1024, 512
    kv_np = lattice_kv(l, N, c, seed=17 + pair[0] * 4 + pair[1])
    src, offsets = oracle.encode_context(kv_np, pair[0])
    want = oracle_transcode_context(src, offsets, [256, 256], [pair[0]] * 2, [pair[1]] * 2, l, c)
    din, _ = kvh.plan_chunks(l, c, N, pair[0])
    dout, total = kvh.plan_chunks(l, c, N, pair[1])
    for hint in (pair, (-1, -1)):
        out = torch.empty(total, dtype=torch.uint8, device="cuda")
        kvh.transcode(torch.from_numpy(src).cuda(), kvh.descs_to_tensor(din, "cuda"), out,
                      kvh.descs_to_tensor(dout, "cuda"), 2, l, c, *hint)
        assert np.array_equal(out.cpu().numpy(), want)
