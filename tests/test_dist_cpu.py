"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, max-over-ranks timing."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2407_20143_b200 import dist
    assert dist.init("gloo")
    rank, _, ws = dist.world()
    dist.barrier()
    agg = dist.aggregate_throughput(units_local=100.0 * (rank + 1), ms_local=10.0 * (rank + 1))
    dist.barrier()
    if rank == 0:
        print(json.dumps(agg))
    dist.shutdown()
""") % ROOT


def test_two_rank_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29600 + os.getpid() % 300
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json

    agg = json.loads(outs[0][0].strip().splitlines()[-1])
    # slowest rank took 20 ms, both ranks together processed 300 units
    assert agg["ms"] == 20.0 and agg["units"] == 300.0 and abs(agg["per_second"] - 15000.0) < 1e-6


def test_single_process_is_a_no_op():
    from paper_2407_20143_b200 import dist

    env_ws = os.environ.pop("WORLD_SIZE", None)
    try:
        assert dist.init() is False
        assert dist.max_over_ranks(3.5) == 3.5
        assert dist.aggregate_throughput(10.0, 5.0)["per_second"] == 2000.0
    finally:
        if env_ws is not None:
            os.environ["WORLD_SIZE"] = env_ws
