"""The multi-rank bookkeeping (replicas only: no collective on the data path) on two CPU ranks
over gloo, and the launch contract of `bench.py --impl reference` under torchrun."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_00061_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r pretends its timed region took 100 + 50 r ms for 10 steps and launched 7 (r + 1) kernels
        ms_local = 100.0 + 50.0 * rank
        value, ms = replicas.aggregate_throughput(10, ms_local)
        mx = replicas.max_over_ranks([ms_local, 1.0 - rank])
        launches = replicas.sum_over_ranks(7 * (rank + 1))
        dist.barrier()
        with open(os.path.join(out_dir, "r%d.json" % rank), "w") as f:
            json.dump(dict(value=value, ms=ms, mx=mx, launches=launches, seed=replicas.rank_seed(0, rank),
                           shard=list(replicas.shard_sequences(5, rank, world))), f)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_totals(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / ("r%d.json" % r))) for r in range(world)]
    for g in got:
        assert g["ms"] == 150.0                              # the slowest rank's time
        assert abs(g["value"] - 2 * 10 / 0.150) < 1e-9       # all ranks' steps over that time
        assert g["mx"] == [150.0, 1.0]
        assert g["launches"] == 7 + 14
    assert got[0]["seed"] != got[1]["seed"]
    assert got[0]["shard"] + got[1]["shard"] == [0, 1, 2, 3, 4]   # every sequence owned exactly once


def test_single_process_needs_no_process_group():
    assert replicas.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert replicas.sum_over_ranks(5) == 5
    value, ms = replicas.aggregate_throughput(10, 100.0)
    assert ms == 100.0 and abs(value - 100.0) < 1e-9
    assert [len(replicas.shard_sequences(7, r, 3)) for r in range(3)] == [2, 2, 3]


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1",
           "--config", "c1"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment spawns two ranks itself
    (rendezvous on 127.0.0.1); with the reference arm rank 0 alone works and prints the line."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "1", "--config", "c1"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2


def test_traffic_record_is_dropped_when_the_kernel_source_changes(tmp_path, monkeypatch):
    import bench
    src = tmp_path / "k.cu"
    src.write_text("v1")
    import hashlib
    rec = {"c2": {"some_kernel": {"traffic_bytes": 123.0, "source_sha256": {"k.cu": hashlib.sha256(b"v1").hexdigest()}}}}
    tf = tmp_path / "traffic.json"
    tf.write_text(json.dumps(rec))
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(tf))
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.ncu_traffic("c2", "some_kernel") == 123.0
    assert bench.ncu_traffic("c3", "some_kernel") is None
    src.write_text("v2")
    assert bench.ncu_traffic("c2", "some_kernel") is None
