"""The multi-rank part of the benchmark (replicas only): times are reduced with
max, work with sum, over a world of 2 gloo ranks on the CPU; and the reference
arm prints only on rank 0."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
r = dist.get_rank()
times, work = bench.reduce_over_ranks(dist, [1.0 + r, 5.0 - r], [10.0 * (r + 1), 7.0, 3.0 + r], torch.device("cpu"))
if r == 0:
    print(json.dumps({"times": times, "work": work, "world": dist.get_world_size()}))
dist.destroy_process_group()
""" % ROOT


def test_replica_aggregation_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29571", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["world"] == 2
    assert d["times"] == [2.0, 5.0]          # max over ranks
    assert d["work"] == [30.0, 14.0, 7.0]    # sum over ranks


def test_reference_arm_prints_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--steps", "1"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_replica_spawner_environment_and_region_count():
    # `bench.py --gpus N` started without torchrun spawns N replicas itself: one rank per GPU,
    # loopback rendezvous, every rank told the world size
    sys.path.insert(0, ROOT)
    import bench
    envs = bench.replica_envs(4, 29999, base_env={"PATH": "/usr/bin", "WORLD_SIZE": "stale"})
    assert [e["RANK"] for e in envs] == ["0", "1", "2", "3"]
    assert [e["LOCAL_RANK"] for e in envs] == ["0", "1", "2", "3"]
    assert all(e["WORLD_SIZE"] == "4" and e["MASTER_ADDR"] == "127.0.0.1" and e["MASTER_PORT"] == "29999"
               and e["PATH"] == "/usr/bin" for e in envs)
    # a short K-step region is repeated until about MIN_TIMED_S has been timed, within the step cap
    assert bench.n_regions_for(33.0, 20) == 13
    assert bench.n_regions_for(330.0, 200) == 2
    assert bench.n_regions_for(5000.0, 200) == 1
    assert bench.n_regions_for(0.1, 20) == 1 + bench.MAX_EXTRA_STEPS // 20


def test_replica_spawner_runs_one_process_per_rank(tmp_path):
    # the spawner itself, with a stand-in script: two processes, ranks 0 and 1, worst exit code returned
    sys.path.insert(0, ROOT)
    import bench
    script = tmp_path / "child.py"
    script.write_text("import os, sys\n"
                      f"open(os.path.join({str(tmp_path)!r}, 'rank' + os.environ['RANK']), 'w').write(os.environ['WORLD_SIZE'])\n"
                      "sys.exit(3 if os.environ['RANK'] == '1' else 0)\n")
    saved = bench.__file__
    bench.__file__ = str(script)
    try:
        rc = bench.spawn_replicas(2, [])
    finally:
        bench.__file__ = saved
    assert rc == 3
    assert (tmp_path / "rank0").read_text() == "2" and (tmp_path / "rank1").read_text() == "2"
