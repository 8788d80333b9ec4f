"""The N>1 path (token sharding + max-over-ranks timing) on two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2510_11370_b200 import dist as r3dist


def test_shard_ranges_cover_everything_once():
    for total in (0, 1, 7, 4096, 4097):
        for world in (1, 2, 3, 8):
            spans = [r3dist.shard_range(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, w = r3dist.init("gloo")
    lo, hi = r3dist.shard_range(1001, r, w)
    r3dist.barrier()
    slowest = r3dist.max_over_ranks(10.0 + r)           # rank 1 is "slower"
    units = r3dist.sum_over_ranks(hi - lo)
    out.put((r, slowest, units))
    torch.distributed.destroy_process_group()


def test_two_ranks_agree_on_job_time_and_total_units():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in res] == [0, 1]
    assert all(r[1] == 11.0 and r[2] == 1001.0 for r in res)


def test_rank_launcher_starts_one_process_per_rank():
    """`bench.py --gpus N` without a launcher environment starts its N ranks through
    dist.run_ranks; the same command line is driven here with a gloo child program."""
    import json
    import subprocess
    child = os.path.join(os.path.dirname(os.path.abspath(__file__)), "dist_child.py")
    cmd = r3dist.launch_command(2, child, ["--gpus", "2", "--units", "77"], r3dist.free_port())
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                  # rank 0 alone prints
    assert lines[0] == {"n_gpus": 2, "asked": 2, "slowest": 11.0, "units": 77.0, "local_rank": 0}


def test_bench_with_a_rank_count_and_no_launcher_starts_the_ranks_itself(monkeypatch):
    import sys
    import pytest
    import bench
    seen = {}

    def fake_run_ranks(n, script, argv, env=None):
        seen.update(n=n, script=script, argv=list(argv))
        return 0

    monkeypatch.setattr(r3dist, "run_ranks", fake_run_ranks)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2", "--warmup", "3"])
    with pytest.raises(SystemExit) as done:
        bench.main()
    assert done.value.code == 0
    assert seen["n"] == 4 and seen["script"].endswith("bench.py")
    assert seen["argv"] == ["--gpus", "4", "--steps", "2", "--warmup", "3"]
