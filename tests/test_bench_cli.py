"""Host-side pieces of bench.py that need no GPU: the policy timing leg, the byte accounting of the
roofline, the issue-rate bound reported for transcoding, and the workload descriptions."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import oracle  # noqa: E402
import workloads  # noqa: E402


def test_policy_leg_prints_one_json_line_and_respects_the_capacity():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--policy-entries", "3000", "--steps", "1"],
                         capture_output=True, text=True, check=True).stdout.strip().splitlines()
    assert len(out) == 1
    r = json.loads(out[0])
    assert r["entries"] == 3000 and r["options_per_entry"] == 16
    assert 0 < r["used_bytes"] <= r["capacity_bytes"]
    assert 0 < r["stored_entries"] <= 3000 and r["value"] > 0


def test_algorithmic_bytes_are_the_stream_plus_two_bytes_per_element():
    """What the roofline divides by the launch time, for one full chunk of the 70B shape at every
    level: the stored size the oracle gives plus 2 bytes per element, i.e. 4, 3.125, 2.625 and 2.375
    bytes per element."""
    l, c, n = 80, 1024, 256
    elements = l * 2 * n * c
    for level, per_element in zip(range(4), (4.0, 3.125, 2.625, 2.375)):
        alg = bench.algorithmic_bytes(elements, oracle.level_bytes(level, l, c, n))
        assert alg == per_element * elements


def test_issue_bound_of_a_transcode_launch():
    """The "alu" roofline: elements x instructions per element over 148 SMs x 4 schedulers x 32 lanes x
    clock.  8 instructions per element of the 70B-shaped context at 2 GHz: 1.134 ms."""
    elements = 80 * 2 * 32768 * 1024
    assert bench.ISSUE_LANES_PER_SM == 128
    bound_ms = elements * 8.0 / (148 * bench.ISSUE_LANES_PER_SM * 2000.0 * 1e3)
    assert bound_ms == pytest.approx(1.1336, rel=1e-3)
    assert set(bench.TRAFFIC["transcode_instr"]) == {(1, 2), (1, 3), (2, 3)}
    assert all(5.0 < v < 12.0 for v in bench.TRAFFIC["transcode_instr"].values())
    assert all(0.9 < v <= 1.0 for kind in ("decode", "encode") for v in bench.TRAFFIC[kind].values())


def test_workload_descriptions():
    names = bench.WORKLOAD_NAMES
    assert names[:5] == ["tiny", "llama3-8b-8k", "batch-64", "llama3-70b-32k", "llama3-8b-128k"]
    c4 = bench.workload_config("llama3-70b-32k")
    assert (c4["n_layers"], c4["n_channels"], c4["n_tokens"], c4["chunk_tokens"], c4["page_tokens"]) == (80, 1024, 32768, 256, 16)
    c3 = bench.workload_config("batch-64")
    assert c3["n_contexts"] == 64 and 64 * workloads.BATCH_MIN_TOKENS <= c3["n_tokens"] <= 64 * workloads.BATCH_MAX_TOKENS
    sliced = bench.workload_config("llama3-70b-32k", tokens=4096)
    assert sliced["n_tokens"] == 4096 and sliced["workload"].endswith("first4096")
    assert len(bench.kernel_source_digest()) == 16
