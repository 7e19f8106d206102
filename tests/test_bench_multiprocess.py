"""The N > 1 host logic of bench.py on CPU: two gloo ranks, replicas only (no data-path collective)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch
    import torch.distributed as dist
    import bench
    rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow replica
    dist.barrier()
    worst = bench.max_over_ranks(dist, ms, torch.device("cpu"))
    assert worst == 15.0, worst
    us = bench.job_us_per_call(worst, 100, world)
    assert abs(us - 15.0 * 1e3 / 200) < 1e-9, us
    # the reference arm runs on rank 0 only; other ranks return without work
    if rank == 1:
        class A: steps = 1; warmup = 0; gpus = world
        assert bench.run_reference(A()) is None
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""") % ROOT


def test_two_gloo_ranks_take_the_slowest_replica(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29631", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for r, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert "rank %d ok" % r in out


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(None, 3.5, None) == 3.5
    assert bench.job_us_per_call(2.0, 10, 1) == 200.0
