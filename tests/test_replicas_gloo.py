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


LAUNCHER = r"""
import sys
sys.path.insert(0, sys.argv[1])
from paper_2401_11504_b200 import runtime
sys.exit(runtime.spawn_replicas([sys.executable, sys.argv[2], sys.argv[1]] + sys.argv[4:], int(sys.argv[3])))
"""


def _launch(tmp_path, worker_src, n, *extra):
    worker, launcher = tmp_path / "worker.py", tmp_path / "launcher.py"
    worker.write_text(worker_src)
    launcher.write_text(LAUNCHER)
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_PORT")}
    return subprocess.run([sys.executable, str(launcher), ROOT, str(worker), str(n), *extra], env=env,
                          capture_output=True, text=True, timeout=300)


def test_spawn_replicas_starts_one_rank_per_gpu_and_passes_rank0_output(tmp_path):
    # what `python bench.py --gpus N` does when it was not started by torch.distributed.run: the same worker as
    # above, started by runtime.spawn_replicas, which picks the port and sets the rank variables itself
    res = _launch(tmp_path, WORKER, 2)
    assert res.returncode == 0, res.stderr[-2000:]
    import json
    lines = [l for l in res.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1                                     # rank 0's line only
    line = json.loads(lines[0])
    assert line["slowest"] == 2.0 and abs(line["value"] - 2 * 10240 / 2.0) < 1e-9


def test_spawn_replicas_reports_a_failing_rank(tmp_path):
    # rank 1 exits with an error before the rendezvous: the launcher ends rank 0 (which would wait for ever)
    # and returns rank 1's code
    failing = "import os, sys, time\nif os.environ['RANK'] == '1':\n    sys.exit(7)\ntime.sleep(120)\n"
    res = _launch(tmp_path, failing, 2)
    assert res.returncode == 7


def test_bench_gpus_n_launches_its_own_workers():
    # without a GPU every worker of `python bench.py --gpus 2` stops at the device check (there is no CPU
    # path): the run must come back promptly with that error, not with a usage message
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for a machine without a GPU")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "2", "--warmup", "1"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode != 0
    assert "needs a CUDA device" in res.stderr and "torch.distributed.run" not in res.stderr


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
