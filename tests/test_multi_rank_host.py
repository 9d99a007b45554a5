"""The only multi-rank logic of the benchmark (replicas only: no data-path collective) is the timing
aggregation: the job's time is the slowest rank's.  Checked with two gloo ranks on CPU."""
import os
import socket
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
