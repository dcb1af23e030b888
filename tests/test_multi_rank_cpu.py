"""The N > 1 path of bench.py on CPU: two `gloo` ranks.  The codec has no exchange step, so the
multi-rank logic is all on the host: every rank works on a context of its own, timings are
combined as the maximum over ranks, the reported value is the whole job's, and the CPU arm
(`--impl reference`) runs on rank 0 alone."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import workloads
    # each rank times its own work: rank r reports (10 + r, 5 - r) milliseconds
    got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], torch.device("cpu"), world)
    kv = workloads.make_kv(1, 32, 32, seed=bench.rank_seed(rank))
    checksum = float(kv.float().sum())
    sums = [None] * world
    dist.all_gather_object(sums, checksum)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"max": got, "sums": sums}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_per_rank_contexts(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        r = json.load(open(tmp_path / f"rank{rank}.json"))
        assert r["max"] == [11.0, 5.0]                    # slowest rank per entry, on every rank
        assert r["sums"][0] != r["sums"][1]               # the ranks drew different contexts


def test_whole_job_value_counts_every_rank():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_gbps(1, 8e9, 2.0)
    assert one == pytest.approx(4000.0)
    assert bench.whole_job_gbps(8, 8e9, 2.0) == pytest.approx(8 * one)      # weak scaling: fixed work per rank
    assert bench.max_over_ranks([1.0, 2.0], torch.device("cpu"), 1) == [1.0, 2.0]


def test_reference_arm_runs_on_rank_zero_only():
    """`torchrun ... bench.py --impl reference --gpus 2`: rank 0 prints the one JSON line, the other
    rank exits 0 without work."""
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference",
           "--gpus", "2", "--steps", "1", "--warmup", "0"]
    env = dict(os.environ, OMP_NUM_THREADS="1")
    p = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["value"] > 0 and out["e2e"]["h2d_bytes_per_step"] == 0


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` without torchrun around it: the script starts two ranks itself (the
    CPU arm here, so no GPU is needed); again one JSON line, from rank 0, for a job of two."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["OMP_NUM_THREADS"] = "1"
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "tiny"]
    p = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["config"]["workload"] == "tiny"


def test_every_workload_has_a_config_without_touching_a_device():
    sys.path.insert(0, ROOT)
    import bench
    names = [bench.workload_config(w)["workload"] for w in bench.WORKLOAD_NAMES]
    assert names == ["tiny", "llama3-8b-8k", "batch-64", "llama3-70b-32k", "llama3-8b-128k"]
    batch = bench.workload_config("batch-64")
    assert batch["n_contexts"] == 64 and 64 * 2048 <= batch["n_tokens"] <= 64 * 32768
    assert bench.workload_config("llama3-70b-32k")["n_tokens"] == 32768
    assert len(bench.kernel_source_digest()) == 16
