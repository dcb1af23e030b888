"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports
every symbol the header declares; the size and layout arithmetic agrees with the
oracle; argument errors are reported without touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kvh():
    from paper_2509_00105_b200 import _build
    _build.build()
    import paper_2509_00105_b200 as k
    k.lib()
    return k


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "kvh.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvh_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(kvh):
    names = declared_symbols()
    assert {"kvh_level_bytes", "kvh_encode", "kvh_decode_to_pages", "kvh_decode_batch"} <= set(names)
    L = ctypes.CDLL(str(kvh.binding._LIB_PATH))
    for n in names:
        assert hasattr(L, n), n


def test_no_environment_variable_steers_the_library():
    """Which kernel runs and how tiles are scheduled is fixed when the library is built: nothing in
    the package reads the process environment."""
    pkg = os.path.join(ROOT, "paper_2509_00105_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")) and f != "_build.py":      # the build script reads NVCC
                text = open(os.path.join(dirpath, f)).read()
                assert "getenv" not in text and "os.environ" not in text, f


def test_build_variants_export_the_same_abi(kvh):
    """The "direct" and "static" builds (other kernels / another tile schedule, chosen at compile
    time) export every declared symbol too and say which build they are; the self-test library
    loads and exports its one entry point."""
    from paper_2509_00105_b200 import _build
    libs = _build.build_all()
    assert kvh.build_variant() == "default"
    for name, want in (("direct", "direct"), ("static", "static-stride")):
        v = kvh.variant(name)
        assert v.build_variant() == want and v is kvh.variant(name)
        L = ctypes.CDLL(str(libs[name]))
        for n in declared_symbols():
            assert hasattr(L, n), (name, n)
    assert kvh.variant("default") is kvh.binding
    with pytest.raises(ValueError):
        kvh.variant("nonesuch")
    assert hasattr(ctypes.CDLL(str(libs["selftest"])), "kvh_selftest_bounded_wait")
    assert hasattr(ctypes.CDLL(str(libs["selftest"])), "kvh_selftest_quanta_ring")


def test_versions_and_level_info(kvh):
    assert kvh.format_version() == 1
    assert kvh.lib().kvh_num_levels() == 4
    assert [kvh.level_info(k) for k in range(4)] == [(16, 0, True), (8, 32, False), (4, 32, False), (2, 32, False)]
    with pytest.raises(kvh.KvhError) as e:
        kvh.level_info(4)
    assert e.value.status == 2
    assert kvh.status_string(6) == "page id outside the pool"


def test_level_bytes_matches_oracle(kvh):
    for l in (1, 3, 32, 80):
        for c in (32, 96, 128, 1024, 4096):
            for n in (1, 2, 15, 16, 17, 31, 32, 33, 64, 100, 255, 256):
                for k in range(4):
                    assert kvh.level_bytes(k, l, c, n) == oracle.level_bytes(k, l, c, n) > 0


@pytest.mark.parametrize("args,status", [
    ((4, 1, 32, 1), 2), ((-1, 1, 32, 1), 2), ((0, 0, 32, 1), 3), ((0, 1, 48, 1), 3),
    ((0, 1, 32, 0), 3), ((0, 1, 32, 257), 3),
])
def test_level_bytes_rejects(kvh, args, status):
    with pytest.raises(kvh.KvhError) as e:
        kvh.level_bytes(*args)
    assert e.value.status == status
    assert oracle.level_bytes(*args) == 0


def test_plan_chunks_matches_oracle(kvh):
    l, c = 4, 64
    for N, levels in [(256, 2), (1000, [0, 1, 2, 3]), (257, [3, 0]), (5, 1), (8192, 3)]:
        descs, total = kvh.plan_chunks(l, c, N, levels, stream_base=256, pt_base=7)
        ntoks, lv, offsets = oracle.chunk_plan(N, levels, l, c)
        assert total == offsets[-1]
        assert descs["stream_off"].tolist() == [256 + o for o in offsets[:-1]]
        assert descs["n_tok"].tolist() == ntoks and descs["level"].tolist() == lv
        assert descs["pt_off"].tolist() == [7 + 16 * i for i in range(len(ntoks))]
        assert not descs["reserved"].any()
    descs, _ = kvh.plan_chunks(l, c, 600, 0, page_tokens=32)
    assert descs["pt_off"].tolist() == [0, 8, 16]


def test_plan_chunks_rejects(kvh):
    for kwargs, status in [(dict(stream_base=64), 4), (dict(page_tokens=24), 3), (dict(pt_base=-1), 1)]:
        with pytest.raises(kvh.KvhError) as e:
            kvh.plan_chunks(2, 64, 300, 1, **kwargs)
        assert e.value.status == status
    with pytest.raises(kvh.KvhError) as e:
        kvh.plan_chunks(2, 64, 300, [1, 9])
    assert e.value.status == 2
    with pytest.raises(ValueError):
        kvh.plan_chunks(2, 64, 300, [1])


def test_device_entry_points_reject_bad_arguments_before_any_cuda_call(kvh):
    L = kvh.lib()
    buf = (ctypes.c_uint8 * 4096)()
    a = (ctypes.addressof(buf) + 127) & ~127          # host memory: never dereferenced on these paths
    assert L.kvh_encode(None, 1, 256, 32, 0, a, 1 << 20, None, None) == 1
    assert L.kvh_encode(a, 1, 0, 32, 0, a, 1 << 20, None, None) == 1
    assert L.kvh_encode(a, 1, 256, 32, 7, a, 1 << 20, None, None) == 2
    assert L.kvh_encode(a, 1, 256, 40, 0, a, 1 << 20, None, None) == 3
    assert L.kvh_encode(a + 8, 1, 256, 32, 0, a, 1 << 20, None, None) == 4
    assert L.kvh_encode(a, 1, 256, 32, 0, a + 64, 1 << 20, None, None) == 4
    assert L.kvh_encode(a, 1, 256, 32, 0, a, 100, None, None) == 5
    assert L.kvh_encode_chunks(a, 1, 600, 32, a, None, 2, a, 1 << 20, None, None) == 3      # 600 tokens = 3 chunks
    pool = kvh.binding._PoolStruct(a, 2 * 8 * 16 * 32, 8 * 16 * 32, 16 * 32, 8, 16, 1, 32)
    assert L.kvh_decode_to_pages(None, 0, 16, a, ctypes.byref(pool), None, None) == 1
    assert L.kvh_decode_to_pages(a, 4, 16, a, ctypes.byref(pool), None, None) == 2
    assert L.kvh_decode_to_pages(a, 0, 300, a, ctypes.byref(pool), None, None) == 3
    assert L.kvh_decode_to_pages(a + 16, 0, 16, a, ctypes.byref(pool), None, None) == 4
    bad = kvh.binding._PoolStruct(a, 2 * 8 * 16 * 32, 8 * 16 * 32, 16 * 32 + 4, 8, 16, 1, 32)
    assert L.kvh_decode_to_pages(a, 0, 16, a, ctypes.byref(bad), None, None) == 4
    bad = kvh.binding._PoolStruct(a, 2 * 8 * 16 * 32, 8 * 16 * 32, 16 * 32, 8, 24, 1, 32)
    assert L.kvh_decode_to_pages(a, 0, 16, a, ctypes.byref(bad), None, None) == 3
    assert L.kvh_decode_batch(a, 4096, None, 1, a, 16, ctypes.byref(pool), None, None) == 1
    assert L.kvh_decode_batch(a, 4096, a, 0, a, 16, ctypes.byref(pool), None, None) == 0   # nothing to do


def test_missing_library_fails_loudly(kvh, monkeypatch, tmp_path):
    from paper_2509_00105_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "libkvh.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_00105_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f


def test_kept_runs_match_the_oracle(kvh):
    import oracle
    for N, a, b in [(1000, 4, 252), (1000, 0, 10), (1000, 10, 0), (100, 60, 40), (100, 80, 40), (5, 0, 0), (7, 7, 0),
                    (1 << 40, 4, 1 << 20)]:
        runs, kept = kvh.keep_sinks_and_recent(N, a, b)
        got = [(int(r["first"]), int(r["count"])) for r in runs]
        if a == 0 and b == 0:
            assert got == [] and kept == 0
            continue
        assert got == oracle.keep_sinks_and_recent(N, a, b)
        assert kept == sum(n for _, n in got)
    with pytest.raises(kvh.KvhError):
        kvh.keep_sinks_and_recent(0, 1, 1)
    with pytest.raises(kvh.KvhError):
        kvh.keep_sinks_and_recent(10, -1, 1)


def test_launches_too_large_for_a_grid_and_new_entry_points_reject_before_any_cuda_call(kvh):
    L = kvh.lib()
    buf = (ctypes.c_uint8 * 4096)()
    a = (ctypes.addressof(buf) + 127) & ~127
    # one CTA per (chunk, layer, K|V, tile): 2^27 chunks x 80 layers x 16 does not fit a grid
    wide = kvh.binding._PoolStruct(a, 2 * 8 * 16 * 32, 8 * 16 * 32, 16 * 32, 8, 16, 80, 32)
    assert L.kvh_decode_batch(a, 1 << 40, a, 1 << 27, a, 1 << 31, ctypes.byref(wide), None, None) == 3
    assert L.kvh_encode(a, 80, (1 << 27) * 256, 32, 3, a, 1 << 60, None, None) == 3
    assert L.kvh_transcode(a, 1 << 40, a, a, 1 << 40, a, None, None, 1 << 27, 80, 32, -1, -1, None, None) == 3
    # transcode: levels, shapes, alignment
    assert L.kvh_transcode(None, 4096, a, a, 4096, a, None, None, 1, 1, 32, -1, -1, None, None) == 1
    assert L.kvh_transcode(a, 4096, a, a, 4096, a, None, None, 1, 1, 32, 2, 1, None, None) == 2
    assert L.kvh_transcode(a, 4096, a, a, 4096, a, None, None, 1, 1, 32, 1, -1, None, None) == 2
    assert L.kvh_transcode(a, 4096, a, a, 4096, a, None, None, 1, 1, 2080, 0, 1, None, None) == 3
    assert L.kvh_transcode(a + 64, 4096, a, a, 4096, a, None, None, 1, 1, 32, 0, 1, None, None) == 4
    assert L.kvh_transcode(a, 4096, a, a, 4096, a, None, None, 0, 1, 32, 0, 1, None, None) == 0      # nothing to do
    # token dropping: runs
    runs = (ctypes.c_int64 * 4)(0, 10, 5, 10)                                     # overlapping
    assert L.kvh_encode_kept(a, 1, 100, 32, runs, 2, a, 1, -1, a, 1 << 20, None, None) == 1
    runs = (ctypes.c_int64 * 2)(0, 10)
    assert L.kvh_encode_kept(a, 1, 100, 32, runs, 1, None, 1, -1, a, 1 << 20, None, None) == 1   # no descriptors, no level
    assert L.kvh_encode_kept(a, 1, 100, 32, runs, 1, None, 2, 1, a, 1 << 20, None, None) == 3    # 10 kept tokens = 1 chunk
    assert L.kvh_encode_kept(a, 1, 100, 32, runs, 1, None, 1, 1, a, 64, None, None) == 5
    assert L.kvh_encode_kept(a, 1, 100, 2080, runs, 1, None, 1, 1, a, 1 << 20, None, None) == 3      # 65 x 32: no block width
    # policy: arguments
    assert L.kvh_policy_assign(None, a, a, 1, a, a, None, None) == 1
    tier = np.array([(1.0, 0.0, 100)], dtype=kvh.TIER_DTYPE)                      # bandwidth must be positive
    freq = np.array([1.0]); opts = np.array([(10, 1.0)], dtype=kvh.OPTION_DTYPE); begin = np.array([0, 1], dtype=np.int32)
    choice = np.zeros(1, dtype=np.int32)
    assert L.kvh_policy_assign(freq.ctypes.data, opts.ctypes.data, begin.ctypes.data, 1, tier.ctypes.data,
                               choice.ctypes.data, None, None) == 1


def test_header_is_plain_c(tmp_path):
    """include/kvh.h is a C header: a C99 compiler takes it with warnings as errors."""
    import subprocess
    src = tmp_path / "use_kvh.c"
    src.write_text('#include "kvh.h"\n'
                   "int main(void) { kvh_token_run r = {0, 1}; kvh_option o = {1, 0.5}; kvh_tier t = {1.0, 1.0, 1};\n"
                   "  kvh_pool p; kvh_chunk_desc d; (void)r; (void)o; (void)t; (void)p; (void)d;\n"
                   "  return kvh_format_version() == KVH_FORMAT_VERSION ? 0 : 1; }\n")
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-fsyntax-only", f"-I{inc}", str(src)],
                   check=True)


def test_page_table_check(kvh):
    import workloads
    t = workloads.shuffled_page_table(500, 600, seed=1).numpy()
    assert kvh.check_page_table(t, 600) == (0, -1)
    u = t.copy(); u[77] = 600
    assert kvh.check_page_table(u, 600) == (6, 77)
    u = t.copy(); u[10] = -1
    assert kvh.check_page_table(u, 600) == (6, 10)
    u = t.copy(); u[300] = u[12]
    assert kvh.check_page_table(u, 600) == (1, 300)
    assert kvh.check_page_table(np.zeros(0, dtype=np.int32), 5) == (0, -1)


def test_ring_of_stage_quanta_never_overlaps_and_never_stalls_empty():
    """The decode kernel cuts its shared-memory stages from a ring of quanta (1 to 3 per unit by
    level, contiguous, taken and given back in order).  The producer's book-keeping is host/device
    code; a test-only entry point (host code, no GPU) drives it with seeded sequences of unit sizes
    against an occupancy map: a unit's quanta must be free when it gets them, lie inside the ring and
    all come back, and an empty ring must take any unit."""
    from paper_2509_00105_b200 import _build
    L = ctypes.CDLL(str(_build.build(variant="selftest")))
    L.kvh_selftest_quanta_ring.restype = ctypes.c_int64
    L.kvh_selftest_quanta_ring.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_uint64, ctypes.POINTER(ctypes.c_int)]
    most = ctypes.c_int(0)
    for n_quanta in (6, 7, 9, 12, 18, 24):                    # 6: rows of 1024 channels; more: narrower rows
        for seed in range(5):
            assert L.kvh_selftest_quanta_ring(n_quanta, 200_000, seed, ctypes.byref(most)) == 0, (n_quanta, seed)
            assert 2 <= most.value <= 8
    assert most.value == 8                                     # 24 quanta: the 8 unit slots are the limit
    assert L.kvh_selftest_quanta_ring(5, 10, 0, None) < 0 and L.kvh_selftest_quanta_ring(25, 10, 0, None) < 0
    assert L.kvh_selftest_quanta_ring(6, 0, 0, ctypes.byref(most)) == 0
