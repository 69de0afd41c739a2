"""The N > 1 path on CPU: N independent replicas, a barrier around the timed region, the
maximum over ranks of the measured time and the sum of the processed units (gloo, world size 2)."""
import os
import subprocess
import sys

from conftest import ROOT

WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
from paper_2401_11504_b200 import runtime
ranks = runtime.Ranks(backend="gloo")
assert ranks.world == 2 and ranks.group
ranks.barrier()
seconds = 0.5 if ranks.rank == 0 else 2.0          # rank 1 is the slow replica
value, slowest = runtime.aggregate_throughput(1024 * 10, seconds, ranks)
assert ranks.max_over_ranks(ranks.rank) == 1.0 and ranks.sum_over_ranks(1.0) == 2.0
ranks.barrier()
if ranks.rank == 0:
    print(json.dumps({"value": value, "slowest": slowest}))
ranks.close()
"""


def test_two_replicas_aggregate_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29547", WORLD_SIZE="2")
    procs = []
    for rank in range(2):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    # both replicas' tokens over the slower replica's time
    assert line["slowest"] == 2.0 and abs(line["value"] - 2 * 10240 / 2.0) < 1e-9


def test_single_process_is_world_size_one():
    from paper_2401_11504_b200 import runtime
    env_backup = {k: os.environ.pop(k, None) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    try:
        ranks = runtime.Ranks()
        assert ranks.world == 1 and not ranks.group
        assert runtime.aggregate_throughput(100, 4.0, ranks) == (25.0, 4.0)
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v
