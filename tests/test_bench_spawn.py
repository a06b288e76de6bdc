"""`bench.py --gpus N` started as a plain process launches its N ranks itself.  Checked here on
CPU with the reference arm (the CPU oracle): two ranks rendezvous over gloo on 127.0.0.1, rank 0
alone computes and prints the one JSON line, which carries n_gpus = 2."""
import json
import os
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def test_bench_gpus_2_spawns_two_ranks_and_prints_one_line():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    env["OMP_NUM_THREADS"] = "4"
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--seq-len", "16"], capture_output=True, text=True, timeout=600, env=env,
                       cwd=str(ROOT))
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert set(d["config"]) >= {"workload", "global_batch", "parallelism"} and "hidden" not in d["config"]


def test_spawn_command_line():
    sys.path.insert(0, str(ROOT))
    import bench
    calls = []
    orig = bench.subprocess.call
    bench.subprocess.call = lambda cmd: calls.append(cmd) or 0
    try:
        assert bench.spawn_ranks(4, ["--gpus", "4", "--steps", "7"]) == 0
    finally:
        bench.subprocess.call = orig
    cmd = calls[0]
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "4", "--steps", "7"]
