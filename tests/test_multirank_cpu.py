"""World-size-2 checks of the benchmark's rank plumbing, on CPU with the gloo backend.

The decode path shards by batch: every rank owns its sequences (own rings, own states) and nothing crosses ranks on
the data path.  What several ranks share is only the measurement: a barrier, the maximum of the per-rank times, and
the whole-job token count.  These tests run that logic in two real processes.
"""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank: int, world: int, port: int, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.rank_env() == (rank, world, rank)
        mine = [[1.0, 5.0], [3.0, 2.0]][rank]
        got = bench.max_over_ranks(mine, dist, "cpu")
        # shards are distinct streams of the same shape
        from ptenc_inputs import CONFIGS, make_inputs
        c = dict(CONFIGS["tiny"])
        k, _ = make_inputs(c, seed=bench.shard_seed(rank)).step_kv(0)
        digest = torch.tensor([float(k.double().sum())], dtype=torch.float64)
        both = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(both, digest)
        dist.barrier()
        q.put((rank, got, [float(x) for x in both], tuple(k.shape)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_own_distinct_shards():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, digests, shape in res:
        assert got == [3.0, 5.0]                       # element-wise max over the two ranks, same on both
        assert digests[0] != digests[1]                # each rank generated its own shard
        assert shape == (1, 2, 1, 64)                  # per-rank batch is the configuration's batch (weak scaling)
    assert res[0][2] == res[1][2]


def test_job_throughput_counts_every_rank():
    import bench
    assert bench.job_tokens_per_s(1, 128, 10, 1000.0) == pytest.approx(1280.0)
    assert bench.job_tokens_per_s(8, 128, 10, 1000.0) == pytest.approx(8 * 1280.0)


def test_reference_arm_under_a_two_rank_launch_prints_once():
    """`bench.py --impl reference` under a two-process launcher: rank 0 times the oracle and prints the line,
    rank 1 exits 0 without output."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference",
           "--gpus", "2", "--steps", "2", "--warmup", "1", "--workload", "tiny"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself():
    """`python bench.py --gpus 2` run directly (no launcher environment) must not quietly run one rank: it re-executes
    itself under the launcher.  Checked with the plumbing-only mode (gloo, no GPU): rank 0 reports two ranks."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR",
                                                              "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--workload", "tiny"],
                       capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(ln) for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1 and lines[0]["dry_run"] and lines[0]["n_gpus"] == 2 and lines[0]["ranks_seen_max_ms"] == 2.0
    assert lines[0]["config"]["parallelism"].startswith("dp2")


def test_gpus_flag_that_disagrees_with_the_launcher_is_an_error():
    env = {**os.environ, "WORLD_SIZE": "1", "RANK": "0", "LOCAL_RANK": "0"}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--dry-run", "--workload", "tiny"],
                       capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert r.returncode != 0 and "launcher started 1 ranks" in r.stderr
