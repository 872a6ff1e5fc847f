"""The reference arm of the benchmark runs without a GPU: it must print one JSON line with the
agreed keys.  (The CUDA arm is exercised on a B200.)"""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl",
                                   "reference", "--steps", "2", "--warmup", "1", "--workload",
                                   "html_tiny"], cwd=ROOT, timeout=600)
    lines = [l for l in out.decode().splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "rows/s" and d["value"] > 0
    assert d["steps"] == 2 and d["warmup"] == 1 and d["higher_is_better"] is True
    assert d["config"]["workload"] == "html_tiny" and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"] == {"value": d["value"], "unit": "rows/s", "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}


def test_other_ranks_of_the_reference_arm_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl",
                                   "reference", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                                  cwd=ROOT, env=env, timeout=600)
    assert out.strip() == b""


def test_gpus_n_without_a_launcher_starts_n_ranks():
    """`bench.py --gpus 2` started plainly must run as two ranks: the launcher command it builds
    is run here on the CPU arm (rank 0 prints the line, rank 1 prints nothing)."""
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl",
                                   "reference", "--steps", "1", "--warmup", "0", "--workload",
                                   "html_tiny", "--gpus", "2"], cwd=ROOT, env=env, timeout=900,
                                  stderr=subprocess.DEVNULL)
    lines = [l for l in out.decode().splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2


def test_spawn_command_names_the_rendezvous_and_passes_the_arguments_on():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.spawn_command(4, ["--gpus", "4", "--steps", "7"], 29511)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-5:] == [os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "7"]
