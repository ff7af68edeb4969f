"""N > 1 runs N independent replicas (the layer has no exchange step).  The only cross-rank logic
is in bench.py: a barrier around the timed region, the maximum of the ranks' times and the sum of
their work.  Checked here with two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    bench._DIST["on"] = True
    bench._DIST["device"] = "cpu"
    rank = dist.get_rank()
    bench.barrier()
    local = 2.0 if rank == 0 else 5.0          # rank 1 is the slow replica
    assert bench.max_over_ranks(local) == 5.0
    v = bench.whole_job_value(dist.get_world_size(), steps=10, units_per_step=3.0, local_seconds=local)
    assert abs(v - 2 * 10 * 3.0 / 5.0) < 1e-12, v
    bench.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""") % ROOT


def test_two_gloo_ranks_aggregate_like_the_bench():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29531", WORLD_SIZE="2")
    procs = []
    for r in range(2):
        e = dict(env, RANK=str(r), LOCAL_RANK=str(r))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, o
        assert f"rank {r} ok" in o


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25) == 1.25
    assert bench.whole_job_value(1, 4, 2.0, 0.5) == 16.0
