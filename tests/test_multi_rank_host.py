"""The only multi-rank logic of the benchmark (replicas only: no data-path collective) is starting the ranks
and the timing aggregation: the job's time is the slowest rank's.  Checked with two gloo ranks on CPU."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    got = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    same = bench.max_over_ranks(3.25, world)
    dist.barrier()
    out.put((rank, got, same))
    dist.destroy_process_group()


def test_time_is_max_over_ranks_gloo_world2():
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
    assert res == [(0, 15.0, 3.25), (1, 15.0, 3.25)]


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.5, 1) == 1.5


def test_reference_arm_runs_on_rank0_only(capsys, monkeypatch):
    sys.path.insert(0, ROOT)
    import bench
    import synthetic as sy
    monkeypatch.setenv("RANK", "1")
    class A: steps, warmup, gpus = 1, 0, 2
    bench.run_reference(A, sy.config_by_name("tiny_fl_fsdp"))
    assert capsys.readouterr().out == ""


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a launcher re-runs itself as two ranks; with the stub workload (no GPU) rank r
    takes 10*(r+1) ms per step, so the line must report two ranks and the slower rank's time."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub-workload", "--steps", "3", "--warmup", "3"],
                         capture_output=True, text=True, cwd=ROOT, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["config"]["parallelism"] == "replicas only" and d["steps"] == 3
    assert abs(d["ms_per_step"] - 20.0) < 1e-9 and abs(d["value"] - 2 * 1000 * 3 / 0.060) < 1e-6


def test_under_a_launcher_the_flag_does_not_spawn_again(monkeypatch):
    sys.path.insert(0, ROOT)
    import bench
    called = []
    monkeypatch.setattr(bench, "spawn_ranks", lambda n, argv: called.append(n) or 0)
    monkeypatch.setattr(bench, "run_stub", lambda args: called.append("stub"))
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--stub-workload"])
    bench.main()
    assert called == ["stub"]
