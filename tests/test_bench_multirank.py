"""N > 1 in the benchmark means independent replicas: the only cross-rank step is aggregating the timing
(max over ranks) and the work (sum over ranks).  Covered with two gloo ranks on CPU, and so is the way
`bench.py --gpus N` starts its N processes by itself."""
import os
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 48.0 * 20, dist, "cpu")
    if rank == 0:
        print(json.dumps({{"ms": ms, "units": units, "world": dist.get_world_size()}}))
    dist.destroy_process_group()
""")


def test_two_rank_aggregation_is_max_time_and_summed_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=str(ROOT)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29541")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res == {"ms": 15.0, "units": 1920.0, "world": 2}


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0) == (3.5, 7.0)


def test_gpus_flag_starts_the_replicas_by_itself():
    """`python bench.py --gpus 2 ...` as ONE plain process (no torchrun, no WORLD_SIZE): it must start two ranks,
    which meet over gloo, and rank 0 alone prints the line, with n_gpus = 2.  The reference arm runs on CPU."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--impl", "reference", "--config", "1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout                       # one line for the whole job
    res = json.loads(lines[0])
    assert res["impl"] == "reference" and res["n_gpus"] == 2 and res["ranks_seen"] == 2
    assert res["value"] > 0 and res["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_under_torchrun_does_not_start_more_processes(monkeypatch):
    sys.path.insert(0, str(ROOT))
    import bench
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("LOCAL_RANK", "1")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2"])
    assert bench.dist_setup(bench.parse_args()) == (2, 1, 1)
