"""The multi-rank plumbing of bench.py on CPU (gloo, world size 2): every rank runs its own replica, the
elapsed time is the maximum over ranks and the reported rate is the whole job's."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import bench
rank, world = bench.dist_init("gloo")
assert world == 2 and rank == int(os.environ["RANK"])
bench.barrier(world)
# rank 1 is the slow one: the job's time is its time
elapsed = bench.max_over_ranks(10.0 if rank == 0 else 25.0, world)
assert elapsed == 25.0, elapsed
rate = bench.whole_job_rate(256, 5, world, elapsed)
assert abs(rate - 256 * 5 * 2 / 0.025) < 1e-6
bench.barrier(world)
if rank == 0:
    print(json.dumps({"elapsed": elapsed, "rate": rate}))
import torch.distributed as dist
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_rank_timing_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = str(_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    assert '"elapsed": 25.0' in outs[0][0]


def test_single_rank_helpers_need_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.0, 1) == 3.0
    assert bench.whole_job_rate(256, 10, 1, 1000.0) == 2560.0
    bench.barrier(1)


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_gpus_flag_without_a_launcher_starts_that_many_ranks():
    """`bench.py --gpus 2` with no launcher in the environment starts two local ranks itself (here only their
    plumbing, on CPU with gloo) and rank 0 reports the world size it actually ran with."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dist-selftest"], env=env,
                         capture_output=True, text=True, timeout=180)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    import json
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2 and rec["requested"] == 2
