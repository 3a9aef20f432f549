"""The N > 1 plumbing of bench.py as two `gloo` processes on CPU: rendezvous on 127.0.0.1 from the launcher's environment
variables, the max over ranks of the timed region, the whole-job value (replicas: weak scaling, no data-path
collective), and the reference arm in which rank 0 alone works and prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(argv_per_rank, world=2, timeout=300):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable] + argv_per_rank, cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=timeout) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    return [o for o, _ in outs]


def test_max_over_ranks_and_whole_job_value_with_gloo():
    code = (
        "import bench, json\n"
        "world, rank, local = bench.dist_setup('gloo')\n"
        "import torch.distributed as dist\n"
        "dist.barrier()\n"
        "ms = bench.max_over_ranks(10.0 * (rank + 1), world, 'cpu')\n"   # rank 1 is the slow one
        "v = bench.whole_job_value(1000, 5, world, ms)\n"
        "print(json.dumps({'rank': rank, 'world': world, 'ms': ms, 'value': v}))\n"
        "dist.destroy_process_group()\n")
    outs = _launch(["-c", code])
    rows = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert sorted(r["rank"] for r in rows) == [0, 1] and all(r["world"] == 2 for r in rows)
    assert all(r["ms"] == 20.0 for r in rows)                      # every rank sees the slowest rank's time
    assert all(abs(r["value"] - 2 * 1000 * 5 / 0.020) < 1e-6 for r in rows)  # whole job = both replicas


def test_single_process_needs_no_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.whole_job_value(100, 2, 1, 1000.0) == 200.0


def test_reference_arm_prints_on_rank_zero_only():
    outs = _launch([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup",
                    "0", "--workload", "c1", "--ref-tokens", "64"])
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert outs[1].strip() == ""


def test_gpus_flag_against_the_launcher_environment():
    """--gpus N either matches the launcher's world size, or (no launcher) makes bench.py start the N ranks itself; a
    contradiction between the two is an error, never a silent single-replica run."""
    import bench
    assert bench.replica_launch_plan(1, {}) == "run"
    assert bench.replica_launch_plan(8, {}) == "spawn"
    assert bench.replica_launch_plan(2, {"WORLD_SIZE": "2"}) == "run"
    assert "contradicts" in bench.replica_launch_plan(8, {"WORLD_SIZE": "2"})
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--impl", "reference"], cwd=ROOT,
                       env=dict(os.environ, WORLD_SIZE="2", RANK="0"), capture_output=True, text=True)
    assert r.returncode != 0 and "contradicts" in r.stderr


def test_reference_arm_covers_training_and_decode_workloads():
    for wl, extra in (("c4", ["--ref-tokens", "1024"]), ("c5-decode", [])):
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                            "--warmup", "0", "--workload", wl] + extra, cwd=ROOT, capture_output=True, text=True,
                           env={k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK")})
        assert r.returncode == 0, r.stderr[-2000:]
        line = json.loads(r.stdout.strip().splitlines()[-1])
        assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["cores"] >= 1
